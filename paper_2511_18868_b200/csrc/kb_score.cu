// kb_score_select: cluster-level statistics, masked-UCB index with the
// Lipschitz term, and arm selection (Sec. 3.4, Assumption 2, Algorithm 1's
// selection line); and the fused tail of a whole step, which prunes (kb_prune's
// arithmetic: roofline floor, saturation mask, gain bound) in the same pass that
// gathers the statistics.
//
//   phase A  score_stats_kernel   one pass over the per-arm history: per-CTA tables of sum(pulls),
//                                 sum(reward_sum) by (strategy, label) and of "any kept member arm" bits in
//                                 shared memory, written out as plain per-CTA partials (no global atomics).
//                                 <PRUNE>: the same pass forms the keep bits and the gain bound of every arm
//                                 from flops / bytes / t_cur and the cluster's saturation bits, so labels and
//                                 keep are read / written once for both calls.
//   phase B  score_table_kernel   adds the partials in CTA order (integer pull totals exact in 64
//                                 bits; the order of the fp32 adds across CTAs is fixed), then
//                                 N, mu, U_cl per (cluster, strategy), the cluster-level argmax and kept_count
//   phase C  score_arms_kernel    per-arm index, mask, optional store, argmax (packed 64-bit atomicMax:
//                                 value, then lowest index); the last CTA of an instance unpacks the keys
// Three launches, no memset node (the first kernel clears the keys the later ones use).
// Streaming traffic: pulls + reward_sum once (8 bytes per arm), labels / dist2 / keep (12 bytes per
// candidate, read by phases A and C), arm_index written once when requested; fused with the pruning:
// + 12 bytes per candidate in, the bound (4 bytes per arm) out.
//
// Measured and not kept for the statistics pass (same results, no faster): a lane per strategy (every access a
// contiguous line and the atomics of a row on consecutive words, but four times the load instructions and half
// the bytes in flight: large 77 against 59 us for the tail, contraction 282 against 189); rows staged through a
// three-stage shared-memory ring by bulk copies, with and without a dedicated copying warp (200 against 192 us on
// contraction before the arms kernel below was reshaped): the pass is bound by its shared-memory atomics, not by
// how its rows arrive -- an fp32 shared-memory atomic add is a compare-and-swap loop (13 cycles per warp
// instruction on random addresses against 3.7 for an integer add, measured alone). Moving the reward sums out
// of shared memory, one four-wide fp32 vector reduction per (row, strategy quad) into a global [K][S] table,
// was slower still (tail 243 against 189 us on contraction, 69 against 59 on large): the table is small, so
// every SM's reductions meet on the same few hundred L2 lines.  Taking a CTA's rows in label order (the counting
// sort of the centroid update, sums of a label's run in registers, the tables touched once per run) lost too:
// the rows of the history are 32 to 128 bytes, the sort and the second look at the labels cost more than the
// atomics they replace (tail 312 against 194 us on contraction, 67 against 59 on large, 30 against 22 on medium).
//
// The shared tables are laid out [strategy][label] with an odd row pitch: the lanes of a warp (a few rows x
// the strategy quads of a row) then fall on different banks unless two rows' labels agree modulo 4, where the
// [label][strategy] layout put every lane that handled the same strategy offset on the same bank.
#include <string.h>

#include "kb_internal.cuh"

namespace {

constexpr int SC_T = 1024;  // threads of the stats kernel (one CTA per SM)

struct ScoreWs {
    unsigned long long* key;    // [B][2]  packed argmax keys: arm level, cluster level
    unsigned* ticket;           // [B]     CTAs of the arms kernel that have finished
    unsigned* part_k;           // [B][G]  per-CTA number of kept arms (fused pruning)
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
    w.ticket = reinterpret_cast<unsigned*>(ws + o);          o += kb_align256((size_t)B * 4);
    w.zero_bytes = o;
    w.part_k = reinterpret_cast<unsigned*>(ws + o);          o += kb_align256((size_t)B * G * 4);
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

// What the fused pruning needs beside the statistics' own inputs (all null / unused without it).
struct PruneIn {
    const float* flops;        // [B][N]
    const float* bytes;        // [B][N]
    const float* t_cur;        // [B][N], needed for the bound only
    const float* peak_flops;   // [S]
    const float* peak_bw;      // [S]
    const float* t_inc;        // [B]
    const float* hsig;         // [B][K][R], null: no saturation mask
    const int32_t* target;     // [S]
    float theta;
    int R;
    uint32_t* keep;            // [B][N] out
    float* bound;              // [B][N][S] out, nullable
};

template <int V, bool PRUNE>
__global__ void __launch_bounds__(SC_T)
score_stats_kernel(int N, int K, int S, int G, int KP, RowWalk wk, const int32_t* __restrict__ labels,
                   const int32_t* __restrict__ pulls, const float* __restrict__ reward_sum,
                   const uint32_t* __restrict__ keep_in, PruneIn pr, int* __restrict__ part_p,
                   float* __restrict__ part_r, unsigned* __restrict__ part_a, unsigned* __restrict__ part_k,
                   unsigned long long* __restrict__ g_key, unsigned* __restrict__ g_ticket,
                   int* __restrict__ dev_status) {
    kb_grid_dependency_wait();
    extern __shared__ __align__(16) unsigned char sraw[];
    int* sp = reinterpret_cast<int*>(sraw);                      // [S][KP] pull sums
    float* sr = reinterpret_cast<float*>(sraw) + S * KP;         // [S][KP] reward sums
    unsigned* sa = reinterpret_cast<unsigned*>(sraw) + 2 * S * KP;   // [K] any kept member arm, bit s
    unsigned* ssat = sa + K;                                     // [K] saturation bits of the cluster (PRUNE)
    __shared__ float s_P[32], s_W[32];
    __shared__ unsigned s_cnt[SC_T / 32];
    const int b = blockIdx.y, g = blockIdx.x, tid = threadIdx.x, lane = tid & 31;
    for (int e = tid; e < 2 * S * KP + K; e += SC_T) sp[e] = 0;  // int 0 == float +0 bit pattern
    if (g == 0 && tid < 2) g_key[2 * b + tid] = 0ull;            // the later kernels' argmax keys and ticket
    if (g == 0 && tid == 2) g_ticket[b] = 0u;
    if (PRUNE) {
        if (tid < S) { s_P[tid] = pr.peak_flops[tid]; s_W[tid] = pr.peak_bw[tid]; }
        // saturation mask of every cluster, once per CTA: bit s = [ h_c[target[s]] < theta ]  (all ones without it)
        for (int j = tid; j < K; j += SC_T) {
            unsigned m = 0xffffffffu;
            if (pr.hsig) {
                m = 0u;
                const float* h = pr.hsig + ((size_t)b * K + j) * pr.R;
                for (int s = 0; s < S; ++s) {
                    int tg = pr.target[s];
                    if (tg < 0 || tg >= pr.R) { atomicOr(dev_status, 2); tg = 0; }
                    if (__ldg(h + tg) < pr.theta) m |= 1u << s;
                }
            }
            ssat[j] = m;
        }
    }
    __syncthreads();
    const int rows_per = (N + G - 1) / G;
    const int r0 = g * rows_per, r1 = min(N, r0 + rows_per);
    const int32_t* lb = labels + (size_t)b * N;
    const int q = tid % wk.vps;
    const bool active = tid < wk.active;
    float rP[V], rW[V];
    float tinc = 0.f;
    if (PRUNE) {
#pragma unroll
        for (int i = 0; i < V; ++i) { rP[i] = 1.f / s_P[q * V + i]; rW[i] = 1.f / s_W[q * V + i]; }
        tinc = pr.t_inc[b];
    }
    unsigned count = 0;
    constexpr int U = PRUNE ? 2 : 4;                             // rows in flight per thread
    // the trip count is the same for every thread of the block (the keep bits of a row are OR-ed across its
    // lanes with shuffles); rows past the end are computed on clamped inputs and dropped
    const int trips = (max(r1 - r0, 0) + U * wk.rstep - 1) / (U * wk.rstep);
    for (int it = 0; it < trips; ++it) {
        const int rb = r0 + tid / wk.vps + it * U * wk.rstep;
        int lab[U];
        int4 pv[U];
        float4 wv[U];
        unsigned bits[U];
        float F[U], Q[U], Tk[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int r = min(rb + u * wk.rstep, r1 - 1);        // clamped: loads stay in range
            const bool live = active && rb + u * wk.rstep < r1;
            lab[u] = -1;
            pv[u] = make_int4(0, 0, 0, 0);
            wv[u] = make_float4(0.f, 0.f, 0.f, 0.f);
            bits[u] = 0;
            F[u] = Q[u] = 0.f; Tk[u] = 1.f;
            if (live) {
                const size_t row = (size_t)b * N + r;
                lab[u] = __ldg(lb + r);
                const size_t off = row * S + (size_t)q * V;
                if (V == 4) {
                    pv[u] = __ldg(reinterpret_cast<const int4*>(pulls + off));
                    wv[u] = __ldg(reinterpret_cast<const float4*>(reward_sum + off));
                } else {
                    pv[u].x = __ldg(pulls + off);
                    wv[u].x = __ldg(reward_sum + off);
                }
                if (PRUNE) {
                    F[u] = __ldg(pr.flops + row);
                    Q[u] = __ldg(pr.bytes + row);
                    if (pr.bound) Tk[u] = __ldg(pr.t_cur + row);
                } else {
                    bits[u] = keep_in ? __ldg(keep_in + row) : 0xffffffffu;
                }
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const bool live = active && rb + u * wk.rstep < r1;
            int lb_ = lab[u];
            const bool lab_ok = lb_ >= 0 && lb_ < K;
            if (live && !lab_ok) atomicOr(dev_status, 1);
            if (PRUNE) {
                // kb_prune's arithmetic.  Quotients by the reciprocal; where that leaves the floor within a few
                // roundings of the incumbent the decision is taken on the correctly rounded quotients instead,
                // so an arm whose floor EQUALS the incumbent is still pruned (strict <), as the definition says.
                if (!lab_ok) lb_ = 0;                                     // kb_prune treats a bad label as cluster 0
                const size_t row = (size_t)b * N + min(rb + u * wk.rstep, r1 - 1);
                const float rT = 1.f / Tk[u];
                unsigned mine = 0;
                float gq[V];
#pragma unroll
                for (int i = 0; i < V; ++i) {
                    float tlb = fmaxf(F[u] * rP[i], Q[u] * rW[i]);
                    if (fabsf(tlb - tinc) <= 2e-6f * tinc)
                        tlb = fmaxf(kb_div_by(F[u], s_P[q * V + i], rP[i]), kb_div_by(Q[u], s_W[q * V + i], rW[i]));
                    if (tlb < tinc) mine |= 1u << (q * V + i);
                    gq[i] = __saturatef(fmaf(-tlb, rT, 1.f));              // clip(1 - T_lb / T_k, 0, 1); NaN -> 0
                }
                mine &= ssat[lb_];
                for (int o = 1; o < wk.vps; o <<= 1) mine |= __shfl_xor_sync(0xffffffffu, mine, o);
                bits[u] = mine;
                if (live) {
                    if (q == 0) { pr.keep[row] = mine; count += __popc(mine); }
                    if (pr.bound) {
                        float* dst = pr.bound + row * S + (size_t)q * V;
                        if (V == 4) *reinterpret_cast<float4*>(dst) = make_float4(gq[0], gq[1 % V], gq[2 % V], gq[3 % V]);
                        else dst[0] = gq[0];
                    }
                }
            }
            if (!live || !lab_ok) continue;
            int* dp = sp + (q * V) * KP + lb_;
            float* dr = sr + (q * V) * KP + lb_;
            if (pv[u].x) atomicAdd(dp, pv[u].x);
            if (wv[u].x != 0.f) atomicAdd(dr, wv[u].x);
            if (V == 4) {
                if (pv[u].y) atomicAdd(dp + KP, pv[u].y);
                if (pv[u].z) atomicAdd(dp + 2 * KP, pv[u].z);
                if (pv[u].w) atomicAdd(dp + 3 * KP, pv[u].w);
                if (wv[u].y != 0.f) atomicAdd(dr + KP, wv[u].y);
                if (wv[u].z != 0.f) atomicAdd(dr + 2 * KP, wv[u].z);
                if (wv[u].w != 0.f) atomicAdd(dr + 3 * KP, wv[u].w);
            }
            // any kept member arm per (cluster, strategy): one 32-bit OR per candidate
            if (q == 0 && bits[u]) atomicOr(&sa[lb_], bits[u]);
        }
    }
    if (PRUNE) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) count += __shfl_xor_sync(0xffffffffu, count, o);
        if (lane == 0) s_cnt[tid >> 5] = count;
    }
    __syncthreads();
    const size_t pbase = ((size_t)b * G + g) * K * S;
    for (int e = tid; e < K * S; e += SC_T) {                    // partials leave as [label][strategy]
        const int cl = e / S, s = e - cl * S;
        part_p[pbase + e] = sp[s * KP + cl];
        part_r[pbase + e] = sr[s * KP + cl];
    }
    for (int j = tid; j < K; j += SC_T) part_a[((size_t)b * G + g) * K + j] = sa[j];
    if (tid == 0) {
        unsigned tot = 0;
        if (PRUNE) for (int w = 0; w < SC_T / 32; ++w) tot += s_cnt[w];
        part_k[(size_t)b * G + g] = tot;
    }
}

constexpr int TB_E = 32, TB_Y = 32;   // entries per block; at most TB_Y slices of the partial index (blockDim.y)   // entries x slices of the partial index per block
__global__ void __launch_bounds__(TB_E * TB_Y)
score_table_kernel(int K, int S, int G, kb_score_params prm, const int32_t* __restrict__ t,
                   const int* __restrict__ part_p, const float* __restrict__ part_r,
                   const unsigned* __restrict__ part_a, float* __restrict__ table, unsigned* __restrict__ anyk,
                   float* __restrict__ cl_pulls, float* __restrict__ cl_mean, float* __restrict__ cl_index,
                   unsigned long long* __restrict__ g_key, const unsigned* __restrict__ part_k,
                   uint32_t* __restrict__ kept_count) {
    kb_grid_dependency_wait();
    if (kept_count && blockIdx.x == 0 && threadIdx.y == 0) {
        // number of kept arms of the instance: the per-CTA counts of the fused pruning, added by one warp
        unsigned c = 0;
        for (int g = threadIdx.x; g < G; g += TB_E) c += part_k[(size_t)blockIdx.y * G + g];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) c += __shfl_xor_sync(0xffffffffu, c, o);
        if (threadIdx.x == 0) kept_count[blockIdx.y] = c;
    }
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

__device__ __forceinline__ void decode_keys(unsigned long long key, unsigned long long ckey, int b,
                                            int32_t* __restrict__ best_arm, float* __restrict__ best_val,
                                            int32_t* __restrict__ best_cluster_arm) {
    if (key == 0) {
        best_arm[b] = -1;
        best_val[b] = -INFINITY;
    } else {
        best_arm[b] = (int32_t)(0xffffffffu - (unsigned)(key & 0xffffffffull));
        best_val[b] = kb_from_orderable((unsigned)(key >> 32));
    }
    best_cluster_arm[b] = ckey ? (int32_t)(0xffffffffu - (unsigned)(ckey & 0xffffffffull)) : -1;
}

constexpr int SA_T = 512;   // threads of the arms kernel

template <int V>
__global__ void __launch_bounds__(SA_T)
score_arms_kernel(int N, int K, int S, int G, RowWalk wk, kb_score_params prm, const int32_t* __restrict__ labels,
                  const float* __restrict__ dist2, const uint32_t* __restrict__ keep,
                  const float* __restrict__ bound, const float* __restrict__ table, float* __restrict__ arm_index,
                  unsigned long long* __restrict__ g_key, unsigned* __restrict__ g_ticket,
                  int32_t* __restrict__ best_arm, float* __restrict__ best_val, int32_t* __restrict__ best_cluster_arm) {
    kb_grid_dependency_wait();
    extern __shared__ __align__(16) float stab[];  // [K][S]
    __shared__ unsigned long long s_best[SA_T / 32];
    const int b = blockIdx.y, tid = threadIdx.x, KS = K * S;
    const int rows_per = (N + G - 1) / G;
    const int r0 = blockIdx.x * rows_per, r1 = min(N, r0 + rows_per);
    const bool cap = prm.cap_with_bound && bound;
    const float L = prm.lipschitz_L;
    unsigned long long best = 0;
    // per thread the arms come in ascending flat index, so a strict comparison keeps the lowest
    // index among equal values; the 64-bit key is built once per thread
    float bestv = -INFINITY;
    unsigned besti = 0xffffffffu;
    const int q = tid % wk.vps;
    constexpr int U = 4;                                           // rows in flight per thread
    int lab[U];
    float d2[U];
    unsigned bits[U];
    float4 bv[U];
    auto request = [&](int rb) {
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int r = min(rb + u * wk.rstep, r1 - 1);          // clamped: loads stay in range
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
    };
    const bool walker = tid < wk.active;
    const int rb0 = r0 + tid / wk.vps;
    // the first rows are requested before the table is staged: their latency runs under the staging
    if (walker && rb0 < r1) request(rb0);
    for (int e = tid; e < KS; e += SA_T) stab[e] = table[(size_t)b * KS + e];
    __syncthreads();
    if (walker) {
        for (int rb = rb0; rb < r1; rb += U * wk.rstep) {
            if (rb != rb0) request(rb);
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
        // the last CTA of the instance to get here unpacks the two keys (its own atomicMax and every earlier
        // CTA's are ordered before its ticket by the fences)
        __threadfence();
        if (atomicAdd(&g_ticket[b], 1u) == (unsigned)G - 1u) {
            __threadfence();
            decode_keys(*reinterpret_cast<volatile unsigned long long*>(&g_key[2 * b]),
                        *reinterpret_cast<volatile unsigned long long*>(&g_key[2 * b + 1]), b, best_arm, best_val,
                        best_cluster_arm);
        }
    }
}

// instances without candidates: nothing ran the arms kernel, the keys are unpacked here
__global__ void score_decode_kernel(int B, const unsigned long long* __restrict__ g_key, int32_t* __restrict__ best_arm,
                                    float* __restrict__ best_val, int32_t* __restrict__ best_cluster_arm) {
    kb_grid_dependency_wait();
    int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= B) return;
    decode_keys(g_key[2 * b], g_key[2 * b + 1], b, best_arm, best_val, best_cluster_arm);
}

}  // namespace

size_t kb_ws_need_score(int B, int N, int K, int S) {
    return carve(nullptr, B, N, K, S).total;
}

static size_t stats_smem(int K, int S, bool prune) {
    const size_t KP = (size_t)(K | 1);
    return (2 * (size_t)S * KP + (prune ? 2 : 1) * (size_t)K) * 4;
}

// The three launches.  pr == nullptr: kb_score_select alone (keep is an input); else the fused tail of a step
// (keep, bound and kept_count are outputs of the first kernel).
static kb_status launch_score_phases(kb_ctx* ctx, int B, int N, int K, int S, kb_score_params p, const int32_t* labels,
                                     const float* dist2, const int32_t* pulls, const float* reward_sum,
                                     const uint32_t* keep, const float* bound, const int32_t* t, float* cl_pulls,
                                     float* cl_mean, float* cl_index, float* arm_index, int32_t* best_arm,
                                     float* best_val, int32_t* best_cluster_arm, const PruneIn* pr, uint32_t* kept_count) {
    const size_t need = kb_ws_need_score(B, N, K, S);
    if (ctx->ws_bytes < need)
        return kb_fail(ctx, KB_ERR_WORKSPACE, "kb_score_select needs %zu bytes of workspace", need);
    ScoreWs w = carve(ctx->ws, B, N, K, S);
    const size_t smem_stats = stats_smem(K, S, pr != nullptr);
    const size_t smem_arms = (size_t)K * S * 4;
    if (smem_stats + 1024 > (size_t)ctx->max_smem_optin)
        return kb_fail(ctx, KB_ERR_UNSUPPORTED, "kb_score_select: K*S = %d is beyond the shared-memory path", K * S);
    // a zero-row instance still gets its (prior-only) tables: run the stats kernel over nothing
    const int G = stats_ctas(B, N, S);
    const int KP = K | 1;
    const bool vec = (S % 4 == 0) && ((((uintptr_t)pulls | (uintptr_t)reward_sum | (uintptr_t)arm_index |
                                        (uintptr_t)bound) & 15) == 0);
    const RowWalk ws_walk = make_walk(SC_T, S, vec ? 4 : 1);
    PruneIn none;
    memset(&none, 0, sizeof(none));
    if (pr) {
        KB_SMEM_OPTIN(ctx, (score_stats_kernel<4, true>), smem_stats);
        kb_launch(score_stats_kernel<4, true>, dim3(G, B), SC_T, smem_stats, ctx->stream, N, K, S, G, KP, ws_walk, labels,
                  pulls, reward_sum, (const uint32_t*)nullptr, *pr, w.part_p, w.part_r, w.part_a, w.part_k, w.key, w.ticket,
                  ctx->dev_status);
    } else if (vec) {
        KB_SMEM_OPTIN(ctx, (score_stats_kernel<4, false>), smem_stats);
        kb_launch(score_stats_kernel<4, false>, dim3(G, B), SC_T, smem_stats, ctx->stream, N, K, S, G, KP, ws_walk, labels,
                  pulls, reward_sum, keep, none, w.part_p, w.part_r, w.part_a, w.part_k, w.key, w.ticket, ctx->dev_status);
    } else {
        KB_SMEM_OPTIN(ctx, (score_stats_kernel<1, false>), smem_stats);
        kb_launch(score_stats_kernel<1, false>, dim3(G, B), SC_T, smem_stats, ctx->stream, N, K, S, G, KP, ws_walk, labels,
                  pulls, reward_sum, keep, none, w.part_p, w.part_r, w.part_a, w.part_k, w.key, w.ticket, ctx->dev_status);
    }
    KB_LAUNCH_CHECK(ctx, "score_stats_kernel");
    const int ty = G >= 64 ? TB_Y : (G >= 8 ? 8 : 1);         // slices of the partial index per entry
    kb_launch(score_table_kernel, dim3((K * S + TB_E - 1) / TB_E, B), dim3(TB_E, ty), 0, ctx->stream,
              K, S, G, p, t, w.part_p, w.part_r, w.part_a, w.table, w.anyk, cl_pulls, cl_mean, cl_index, w.key, w.part_k,
              pr ? kept_count : (uint32_t*)nullptr);
    KB_LAUNCH_CHECK(ctx, "score_table_kernel");
    if (N > 0) {
        long want = (2L * ctx->sm_count + B - 1) / B;               // two CTAs per SM in all
        long capg = ((long)N * S + 4095) / 4096;
        int GA = (int)(want < 1 ? 1 : (want > capg ? capg : want));
        if (GA < 1) GA = 1;
        const RowWalk wa = make_walk(SA_T, S, vec ? 4 : 1);
        const uint32_t* keep_c = pr ? pr->keep : keep;
        if (vec) {
            KB_SMEM_OPTIN(ctx, score_arms_kernel<4>, smem_arms);
            kb_launch(score_arms_kernel<4>, dim3(GA, B), SA_T, smem_arms, ctx->stream, N, K, S, GA, wa, p, labels, dist2,
                      keep_c, bound, w.table, arm_index, w.key, w.ticket, best_arm, best_val, best_cluster_arm);
        } else {
            KB_SMEM_OPTIN(ctx, score_arms_kernel<1>, smem_arms);
            kb_launch(score_arms_kernel<1>, dim3(GA, B), SA_T, smem_arms, ctx->stream, N, K, S, GA, wa, p, labels, dist2,
                      keep_c, bound, w.table, arm_index, w.key, w.ticket, best_arm, best_val, best_cluster_arm);
        }
        KB_LAUNCH_CHECK(ctx, "score_arms_kernel");
    } else {
        kb_launch(score_decode_kernel, (B + 255) / 256, 256, 0, ctx->stream, B, w.key, best_arm, best_val, best_cluster_arm);
        KB_LAUNCH_CHECK(ctx, "score_decode_kernel");
    }
    return KB_OK;
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
    return launch_score_phases(ctx, B, N, K, S, p, labels, dist2, pulls, reward_sum, keep, bound, t, cl_pulls, cl_mean,
                               cl_index, arm_index, best_arm, best_val, best_cluster_arm, nullptr, nullptr);
}

// ---- the fused tail of a whole step: kb_prune and kb_score_select in three launches ------------------------
bool kb_step_tail_fused_eligible(const kb_ctx* ctx, const kb_step_args* a) {
    if (a->B < 1 || a->N < 1 || a->K < 1 || a->R < 1) return false;
    if (a->S != 4 && a->S != 8 && a->S != 16 && a->S != 32) return false;
    if ((long long)a->N * a->S > 0x7fffffffLL) return false;
    if (stats_smem(a->K, a->S, true) + 1024 > (size_t)ctx->max_smem_optin) return false;
    if (!a->flops || !a->bytes || !a->peak_flops || !a->peak_bw || !a->t_incumbent || !a->t_cur || !a->labels ||
        !a->hsig || !a->target || !a->pulls || !a->reward_sum || !a->t || !a->keep || !a->kept_count || !a->cl_pulls ||
        !a->cl_mean || !a->cl_index || !a->best_arm || !a->best_val || !a->best_cluster_arm)
        return false;
    if (a->score.lipschitz_L != 0.f && !a->dist2) return false;
    if (!(a->score.prior_pulls > 0.f)) return false;
    if (a->score.cap_with_bound && !a->bound) return false;
    const uintptr_t al = (uintptr_t)a->pulls | (uintptr_t)a->reward_sum | (uintptr_t)a->bound | (uintptr_t)a->arm_index;
    return (al & 15) == 0;
}

// bound_done: a->bound already holds the gain bound (the host-buffer step computes it early): it is not rewritten
kb_status kb_launch_step_tail_fused(kb_ctx* ctx, const kb_step_args* a, bool bound_done) {
    PruneIn pr;
    pr.flops = a->flops; pr.bytes = a->bytes; pr.t_cur = a->t_cur; pr.peak_flops = a->peak_flops; pr.peak_bw = a->peak_bw;
    pr.t_inc = a->t_incumbent; pr.hsig = a->hsig; pr.target = a->target; pr.theta = a->theta_sat; pr.R = a->R;
    pr.keep = a->keep; pr.bound = bound_done ? nullptr : a->bound;
    return launch_score_phases(ctx, a->B, a->N, a->K, a->S, a->score, a->labels, a->dist2, a->pulls, a->reward_sum,
                               nullptr, a->bound, a->t, a->cl_pulls, a->cl_mean, a->cl_index, a->arm_index, a->best_arm,
                               a->best_val, a->best_cluster_arm, &pr, a->kept_count);
}
