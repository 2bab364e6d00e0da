// kb_score_select: cluster-level statistics, masked-UCB index with the
// Lipschitz term, and arm selection (Sec. 3.4, Assumption 2, Algorithm 1's
// selection line).
//
//   phase A  score_stats_kernel   per-CTA tables of sum(pulls), sum(reward_sum) by (label, s) and of
//                                 "any kept member arm" bits, built with shared-memory atomics and
//                                 written out as plain per-CTA partials (no global atomics)
//   phase B  score_table_kernel   adds the partials in CTA order (integer pull totals exact in 64
//                                 bits; the order of the fp32 adds across CTAs is fixed), then
//                                 N, mu, U_cl per (cluster, strategy) and the cluster-level argmax
//   phase C  score_arms_kernel    per-arm index, mask, optional store, argmax
//                                 (packed 64-bit atomicMax: value, then lowest index)
//   phase D  score_decode_kernel  unpacks the two argmax keys
// Streaming traffic: pulls + reward_sum once (8 bytes per arm), labels / dist2 / keep (12 bytes per
// candidate, read by phases A and C), arm_index written once when requested.
#include "kb_internal.cuh"

namespace {

constexpr int SC_T = 512;   // threads of the stats kernel

struct ScoreWs {
    unsigned long long* key;    // [B][2]  packed argmax keys: arm level, cluster level
    float* table;               // [B][K][S]   U_cl in fp32
    unsigned* anyk;             // [B][K]      any kept member arm, bit s
    int* part_p;                // [B][G][K][S] per-CTA pull sums
    float* part_r;              // [B][G][K][S] per-CTA reward sums
    unsigned* part_a;           // [B][G][K]    per-CTA any-kept bits
    size_t zero_bytes;          // leading bytes that must be cleared per call
    size_t total;
};

int stats_ctas(int B, int N, int S) {
    // about one CTA per SM of a 148-SM part in total, each with at least 4096 arms
    long want = (148 + (long)B - 1) / B;
    long cap = ((long)N * S + 4095) / 4096;
    long g = want < cap ? want : cap;
    return (int)(g < 1 ? 1 : g);
}

ScoreWs carve(char* ws, int B, int N, int K, int S) {
    ScoreWs w;
    const size_t G = stats_ctas(B, N, S);
    size_t o = 0;
    w.key = reinterpret_cast<unsigned long long*>(ws + o);   o += kb_align256((size_t)B * 16);
    w.zero_bytes = o;
    w.table = reinterpret_cast<float*>(ws + o);              o += kb_align256((size_t)B * K * S * 4);
    w.anyk = reinterpret_cast<unsigned*>(ws + o);            o += kb_align256((size_t)B * K * 4);
    w.part_p = reinterpret_cast<int*>(ws + o);               o += kb_align256((size_t)B * G * K * S * 4);
    w.part_r = reinterpret_cast<float*>(ws + o);             o += kb_align256((size_t)B * G * K * S * 4);
    w.part_a = reinterpret_cast<unsigned*>(ws + o);          o += kb_align256((size_t)B * G * K * 4);
    w.total = o;
    return w;
}

// Thread geometry for walking an [rows][S] array in vectors of V with a fixed strategy offset per
// thread and no division in the loop: T = (threads / vps) * vps threads are active, thread t owns
// vector (t % vps) of rows t / vps, t / vps + T / vps, ...
struct RowWalk {
    int vps;     // vectors per row (S / V)
    int active;  // active threads
    int rstep;   // rows advanced per iteration
};
RowWalk make_walk(int threads, int S, int V) {
    RowWalk w;
    w.vps = S / V;
    w.rstep = threads / w.vps;
    w.active = w.rstep * w.vps;
    return w;
}

template <int V>
__global__ void __launch_bounds__(SC_T)
score_stats_kernel(int N, int K, int S, int G, RowWalk wk, const int32_t* __restrict__ labels,
                   const int32_t* __restrict__ pulls, const float* __restrict__ reward_sum,
                   const uint32_t* __restrict__ keep, int* __restrict__ part_p, float* __restrict__ part_r,
                   unsigned* __restrict__ part_a, int* __restrict__ dev_status) {
    kb_grid_dependency_wait();
    extern __shared__ __align__(16) unsigned char sraw[];
    const int KS = K * S;
    int* sp = reinterpret_cast<int*>(sraw);                      // [K][S]
    float* sr = reinterpret_cast<float*>(sraw) + KS;             // [K][S]
    unsigned* sa = reinterpret_cast<unsigned*>(sraw) + 2 * KS;   // [K]
    const int b = blockIdx.y, g = blockIdx.x, tid = threadIdx.x;
    for (int e = tid; e < 2 * KS + K; e += SC_T) sp[e] = 0;      // int 0 == float +0 bit pattern
    __syncthreads();
    const int rows_per = (N + G - 1) / G;
    const int r0 = g * rows_per, r1 = min(N, r0 + rows_per);
    const int32_t* lb = labels + (size_t)b * N;
    if (tid < wk.active) {
        const int q = tid % wk.vps;
        constexpr int U = 4;                                       // rows in flight per thread
        for (int rb = r0 + tid / wk.vps; rb < r1; rb += U * wk.rstep) {
            int lab[U];
            int4 pv[U];
            float4 wv[U];
            unsigned bits[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int r = rb + u * wk.rstep;
                lab[u] = -1;
                pv[u] = make_int4(0, 0, 0, 0);
                wv[u] = make_float4(0.f, 0.f, 0.f, 0.f);
                bits[u] = 0;
                if (r < r1) {
                    lab[u] = __ldg(lb + r);
                    const size_t off = ((size_t)b * N + r) * S + (size_t)q * V;
                    if (V == 4) {
                        pv[u] = __ldg(reinterpret_cast<const int4*>(pulls + off));
                        wv[u] = __ldg(reinterpret_cast<const float4*>(reward_sum + off));
                    } else {
                        pv[u].x = __ldg(pulls + off);
                        wv[u].x = __ldg(reward_sum + off);
                    }
                    if (q == 0) bits[u] = keep ? __ldg(keep + (size_t)b * N + r) : 0xffffffffu;
                }
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                if (rb + u * wk.rstep >= r1) break;
                if (lab[u] < 0 || lab[u] >= K) { atomicOr(dev_status, 1); continue; }
                int* dp = sp + lab[u] * S + q * V;
                float* dr = sr + lab[u] * S + q * V;
                if (pv[u].x) atomicAdd(dp + 0, pv[u].x);
                if (wv[u].x != 0.f) atomicAdd(dr + 0, wv[u].x);
                if (V == 4) {
                    if (pv[u].y) atomicAdd(dp + 1, pv[u].y);
                    if (pv[u].z) atomicAdd(dp + 2, pv[u].z);
                    if (pv[u].w) atomicAdd(dp + 3, pv[u].w);
                    if (wv[u].y != 0.f) atomicAdd(dr + 1, wv[u].y);
                    if (wv[u].z != 0.f) atomicAdd(dr + 2, wv[u].z);
                    if (wv[u].w != 0.f) atomicAdd(dr + 3, wv[u].w);
                }
                // any kept member arm per (cluster, strategy): one 32-bit OR per candidate
                if (q == 0 && bits[u]) atomicOr(&sa[lab[u]], bits[u]);
            }
        }
    }
    __syncthreads();
    const size_t pbase = ((size_t)b * G + g) * KS;
    for (int e = tid; e < KS; e += SC_T) { part_p[pbase + e] = sp[e]; part_r[pbase + e] = sr[e]; }
    for (int j = tid; j < K; j += SC_T) part_a[((size_t)b * G + g) * K + j] = sa[j];
}

constexpr int TB_E = 32, TB_Y = 32;   // entries per block; at most TB_Y slices of the partial index (blockDim.y)   // entries x slices of the partial index per block
__global__ void __launch_bounds__(TB_E * TB_Y)
score_table_kernel(int K, int S, int G, kb_score_params prm, const int32_t* __restrict__ t,
                   const int* __restrict__ part_p, const float* __restrict__ part_r,
                   const unsigned* __restrict__ part_a, float* __restrict__ table, unsigned* __restrict__ anyk,
                   float* __restrict__ cl_pulls, float* __restrict__ cl_mean, float* __restrict__ cl_index,
                   unsigned long long* __restrict__ g_key) {
    kb_grid_dependency_wait();
    __shared__ long long s_np[TB_Y][TB_E];
    __shared__ float s_rs[TB_Y][TB_E];
    __shared__ unsigned s_any[TB_Y][TB_E];
    const int b = blockIdx.y, x = threadIdx.x, y = threadIdx.y, KS = K * S;
    const int e = blockIdx.x * TB_E + x;
    // slice y adds the partials of CTAs [y*per, (y+1)*per) in order; the slices are then added in order
    const int ny = (int)blockDim.y;
    const int per = (G + ny - 1) / ny;
    long long np_ = 0;
    float rs = 0.f;
    unsigned any = 0;
    if (e < KS) {
        const int cl = e / S;
        const int g1 = min(G, (y + 1) * per);
#pragma unroll 4
        for (int g = y * per; g < g1; ++g) {
            const size_t o = ((size_t)b * G + g) * KS + e;
            np_ += part_p[o];
            rs += part_r[o];
            any |= part_a[((size_t)b * G + g) * K + cl];
        }
    }
    s_np[y][x] = np_; s_rs[y][x] = rs; s_any[y][x] = any;
    __syncthreads();
    unsigned long long best = 0;
    if (y == 0) {
        if (e < KS) {
            for (int k = 1; k < ny; ++k) { np_ += s_np[k][x]; rs += s_rs[k][x]; any |= s_any[k][x]; }
            const int cl = e / S, s = e - cl * S;
            const float lnt = logf((float)t[b]);
            const size_t i = (size_t)b * KS + e;
            // integer total converted once, prior added last
            const float n = prm.prior_pulls + (float)np_;
            const float mu = (prm.prior_pulls * prm.prior_mean + rs) / n;
            const float u = mu + prm.c * sqrtf(lnt / n);
            cl_pulls[i] = n;
            cl_mean[i] = mu;
            cl_index[i] = u;
            table[i] = u;
            if (s == 0) anyk[(size_t)b * K + cl] = any;
            if ((any >> s) & 1u) best = ((unsigned long long)kb_orderable(u) << 32) | (0xffffffffu - (unsigned)e);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            unsigned long long other = __shfl_xor_sync(0xffffffffu, best, o);
            best = other > best ? other : best;
        }
        if (x == 0 && best) atomicMax(&g_key[2 * b + 1], best);
    }
}

template <int V>
__global__ void __launch_bounds__(256)
score_arms_kernel(int N, int K, int S, int G, RowWalk wk, kb_score_params prm, const int32_t* __restrict__ labels,
                  const float* __restrict__ dist2, const uint32_t* __restrict__ keep,
                  const float* __restrict__ bound, const float* __restrict__ table, float* __restrict__ arm_index,
                  unsigned long long* __restrict__ g_key) {
    kb_grid_dependency_wait();
    extern __shared__ __align__(16) float stab[];  // [K][S]
    __shared__ unsigned long long s_best[8];
    const int b = blockIdx.y, tid = threadIdx.x, KS = K * S;
    for (int e = tid; e < KS; e += blockDim.x) stab[e] = table[(size_t)b * KS + e];
    __syncthreads();
    const int rows_per = (N + G - 1) / G;
    const int r0 = blockIdx.x * rows_per, r1 = min(N, r0 + rows_per);
    const bool cap = prm.cap_with_bound && bound;
    const float L = prm.lipschitz_L;
    unsigned long long best = 0;
    // per thread the arms come in ascending flat index, so a strict comparison keeps the lowest
    // index among equal values; the 64-bit key is built once per thread
    float bestv = -INFINITY;
    unsigned besti = 0xffffffffu;
    if (tid < wk.active) {
        const int q = tid % wk.vps;
        constexpr int U = 4;                                       // rows in flight per thread
        for (int rb = r0 + tid / wk.vps; rb < r1; rb += U * wk.rstep) {
            int lab[U];
            float d2[U];
            unsigned bits[U];
            float4 bv[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int r = min(rb + u * wk.rstep, r1 - 1);      // clamped: loads stay in range
                const size_t row = (size_t)b * N + r;
                lab[u] = __ldg(labels + row);
                d2[u] = L != 0.f ? __ldg(dist2 + row) : 0.f;
                bits[u] = keep ? __ldg(keep + row) : 0xffffffffu;
                bv[u] = make_float4(0.f, 0.f, 0.f, 0.f);
                if (cap) {
                    const size_t off = row * S + (size_t)q * V;
                    if (V == 4) bv[u] = __ldg(reinterpret_cast<const float4*>(bound + off));
                    else bv[u].x = __ldg(bound + off);
                }
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int r = rb + u * wk.rstep;
                if (r >= r1) break;
                const int lb_ = lab[u] < 0 ? 0 : (lab[u] >= K ? K - 1 : lab[u]);
                const float smooth = L != 0.f ? L * sqrtf(d2[u]) : 0.f;
                const size_t off = ((size_t)b * N + r) * S + (size_t)q * V;
                float uu[V];
                if (V == 4) {
                    const float4 tv = *reinterpret_cast<const float4*>(stab + lb_ * S + q * V);
                    uu[0] = tv.x + smooth; uu[1 % V] = tv.y + smooth; uu[2 % V] = tv.z + smooth; uu[3 % V] = tv.w + smooth;
                    if (cap) {
                        uu[0] = fminf(uu[0], bv[u].x); uu[1 % V] = fminf(uu[1 % V], bv[u].y);
                        uu[2 % V] = fminf(uu[2 % V], bv[u].z); uu[3 % V] = fminf(uu[3 % V], bv[u].w);
                    }
                } else {
                    uu[0] = stab[lb_ * S + q] + smooth;
                    if (cap) uu[0] = fminf(uu[0], bv[u].x);
                }
                const unsigned flat0 = (unsigned)(r * S + q * V);
#pragma unroll
                for (int i = 0; i < V; ++i) {
                    const bool ok = (bits[u] >> (q * V + i)) & 1u;
                    if (ok) {
                        // (a NaN index never compares greater; -inf is taken when nothing was seen yet)
                        if (uu[i] > bestv || besti == 0xffffffffu) { bestv = uu[i]; besti = flat0 + i; }
                    } else {
                        uu[i] = -INFINITY;
                    }
                }
                if (arm_index) {
                    if (V == 4)
                        *reinterpret_cast<float4*>(arm_index + off) = make_float4(uu[0], uu[1 % V], uu[2 % V], uu[3 % V]);
                    else
                        arm_index[off] = uu[0];
                }
            }
        }
    }
    if (besti != 0xffffffffu) best = ((unsigned long long)kb_orderable(bestv) << 32) | (0xffffffffu - besti);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        unsigned long long other = __shfl_xor_sync(0xffffffffu, best, o);
        best = other > best ? other : best;
    }
    if ((tid & 31) == 0) s_best[tid >> 5] = best;
    __syncthreads();
    if (tid == 0) {
        for (int w = 1; w < (int)(blockDim.x >> 5); ++w) best = s_best[w] > best ? s_best[w] : best;
        if (best) atomicMax(&g_key[2 * b], best);
    }
}

__global__ void score_decode_kernel(int B, const unsigned long long* __restrict__ g_key, int32_t* __restrict__ best_arm,
                                    float* __restrict__ best_val, int32_t* __restrict__ best_cluster_arm) {
    kb_grid_dependency_wait();
    int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= B) return;
    const unsigned long long key = g_key[2 * b], ckey = g_key[2 * b + 1];
    if (key == 0) {
        best_arm[b] = -1;
        best_val[b] = -INFINITY;
    } else {
        best_arm[b] = (int32_t)(0xffffffffu - (unsigned)(key & 0xffffffffull));
        best_val[b] = kb_from_orderable((unsigned)(key >> 32));
    }
    best_cluster_arm[b] = ckey ? (int32_t)(0xffffffffu - (unsigned)(ckey & 0xffffffffull)) : -1;
}

}  // namespace

size_t kb_ws_need_score(int B, int N, int K, int S) {
    return carve(nullptr, B, N, K, S).total;
}

kb_status kb_launch_score(kb_ctx* ctx, int B, int N, int K, int S, kb_score_params p, const int32_t* labels,
                          const float* dist2, const int32_t* pulls, const float* reward_sum, const uint32_t* keep,
                          const float* bound, const int32_t* t, float* cl_pulls, float* cl_mean, float* cl_index,
                          float* arm_index, int32_t* best_arm, float* best_val, int32_t* best_cluster_arm) {
    if (B == 0) return KB_OK;
    if (kb_score_small_eligible(ctx, B, N, K, S, p, dist2, pulls, reward_sum, bound, arm_index))
        // at most 1024 candidates per instance: one CTA per instance does all four phases in one launch
        return kb_launch_score_small(ctx, B, N, K, S, p, labels, dist2, pulls, reward_sum, keep, bound, t, cl_pulls, cl_mean,
                                     cl_index, arm_index, best_arm, best_val, best_cluster_arm);
    const size_t need = kb_ws_need_score(B, N, K, S);
    if (ctx->ws_bytes < need)
        return kb_fail(ctx, KB_ERR_WORKSPACE, "kb_score_select needs %zu bytes of workspace", need);
    ScoreWs w = carve(ctx->ws, B, N, K, S);
    KB_MEMSET(ctx, ctx->ws, 0, w.zero_bytes);
    const size_t smem_stats = ((size_t)2 * K * S + K) * 4;
    const size_t smem_arms = (size_t)K * S * 4;
    if (smem_stats + 1024 > (size_t)ctx->max_smem_optin)
        return kb_fail(ctx, KB_ERR_UNSUPPORTED, "kb_score_select: K*S = %d is beyond the shared-memory path", K * S);
    // a zero-row instance still gets its (prior-only) tables: run the stats kernel over nothing
    const int G = stats_ctas(B, N, S);
    const bool vec = (S % 4 == 0) && ((((uintptr_t)pulls | (uintptr_t)reward_sum | (uintptr_t)arm_index |
                                        (uintptr_t)bound) & 15) == 0);
    const RowWalk ws_walk = make_walk(SC_T, S, vec ? 4 : 1);
    if (vec) {
        KB_SMEM_OPTIN(ctx, score_stats_kernel<4>, smem_stats);
        kb_launch(score_stats_kernel<4>, dim3(G, B), SC_T, smem_stats, ctx->stream, 
            N, K, S, G, ws_walk, labels, pulls, reward_sum, keep, w.part_p, w.part_r, w.part_a, ctx->dev_status);
    } else {
        KB_SMEM_OPTIN(ctx, score_stats_kernel<1>, smem_stats);
        kb_launch(score_stats_kernel<1>, dim3(G, B), SC_T, smem_stats, ctx->stream, 
            N, K, S, G, ws_walk, labels, pulls, reward_sum, keep, w.part_p, w.part_r, w.part_a, ctx->dev_status);
    }
    KB_LAUNCH_CHECK(ctx, "score_stats_kernel");
    const int ty = G >= 64 ? TB_Y : (G >= 8 ? 8 : 1);         // slices of the partial index per entry
    kb_launch(score_table_kernel, dim3((K * S + TB_E - 1) / TB_E, B), dim3(TB_E, ty), 0, ctx->stream, 
        K, S, G, p, t, w.part_p, w.part_r, w.part_a, w.table, w.anyk, cl_pulls, cl_mean, cl_index, w.key);
    KB_LAUNCH_CHECK(ctx, "score_table_kernel");
    if (N > 0) {
        long want = (4L * ctx->sm_count + B - 1) / B;
        long capg = ((long)N * S + 2047) / 2048;
        int GA = (int)(want < 1 ? 1 : (want > capg ? capg : want));
        if (GA < 1) GA = 1;
        const RowWalk wa = make_walk(256, S, vec ? 4 : 1);
        if (vec) {
            KB_SMEM_OPTIN(ctx, score_arms_kernel<4>, smem_arms);
            kb_launch(score_arms_kernel<4>, dim3(GA, B), 256, smem_arms, ctx->stream, 
                N, K, S, GA, wa, p, labels, dist2, keep, bound, w.table, arm_index, w.key);
        } else {
            KB_SMEM_OPTIN(ctx, score_arms_kernel<1>, smem_arms);
            kb_launch(score_arms_kernel<1>, dim3(GA, B), 256, smem_arms, ctx->stream, 
                N, K, S, GA, wa, p, labels, dist2, keep, bound, w.table, arm_index, w.key);
        }
        KB_LAUNCH_CHECK(ctx, "score_arms_kernel");
    }
    kb_launch(score_decode_kernel, (B + 255) / 256, 256, 0, ctx->stream, B, w.key, best_arm, best_val, best_cluster_arm);
    KB_LAUNCH_CHECK(ctx, "score_decode_kernel");
    return KB_OK;
}
