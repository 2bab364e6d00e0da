// kb_cluster_fit for one mid-sized instance: the whole Lloyd loop in ONE cooperative launch.
//
// Between the instances that fit a single CTA (kb_fit_fused.cu) and those large enough for the
// tensor-core kernel lies the launch-latency regime: with N of a few ten thousand rows an
// assign or an update moves about a megabyte, so an iteration of several dependent launches is
// all launch gaps.  Here every CTA keeps its share of the rows on chip (registers and shared
// memory) for all iterations and the CTAs meet once per iteration at a grid-wide barrier:
//   * assign: a thread owns two rows in registers and scans a part of the centroids in shared memory
//     (the threads that share a row each take a contiguous part, the best over the parts is taken
//     in ascending order);
//     the distance is the direct form sum (z - c)^2, ascending centroid id, strict < (lowest id
//     on ties) -- the same arithmetic as the row-wise assign kernel;
//   * update: the CTA's rows are added into a (cluster, column) table in shared memory (a warp adds
//     consecutive columns of one row: conflict-free), then one reduction per (cluster, column) of a
//     non-empty cluster into a global table;
//   * grid barrier (a monotone arrival counter; the launch is cooperative, so all CTAs are
//     resident; the wait is bounded and raises the device status word when it expires);
//   * every CTA reads the table back and forms the new centroids itself.
// The global table is triple-buffered: iteration i accumulates into table i % 3, table
// (i + 1) % 3 is cleared before barrier i, and nobody reads table (i - 2) % 3 any more.  Each table
// is kept in CF_NC copies (CTA g adds into copy g % CF_NC and the readers add the copies up): all
// CTAs reduce into the same few lines, and the reductions on one line are serviced one at a time.
// Z is read from HBM exactly once per fit.
//
// The whole-step drivers hand this kernel the RAW features instead (`xraw`): it then also does what
// kb_normalize and kb_init_centroids would have done.  Every CTA adds up its rows per column (shifted
// by the instance's first row, in double) and stores the partial sums; after one more grid barrier
// every CTA adds all partials in CTA order (so all of them, and every run, get the same statistics),
// normalises its rows in shared memory with kb_normalize's expression and writes z once.  The rows
// that seed the centroids are fetched raw BEFORE that barrier (z may overwrite x in place) and
// normalised with the same expression afterwards.
#include "kb_internal.cuh"

namespace {

constexpr int CF_MAXROWS = 512;    // rows per CTA at most
constexpr int CF_R = 2;            // rows per thread
// threads per CTA: the register file holds CF_R rows of D floats per thread for this many
__host__ __device__ constexpr int cf_threads(int D) { return D <= 32 ? 512 : 256; }
constexpr int CF_NC = 4;           // copies of the global table: CTA g adds into copy g % CF_NC
constexpr unsigned CF_SPIN_LIMIT = 1u << 22;
constexpr int CF_STATUS_TIMEOUT = 0x200;

struct CoopScratch {               // device scratch, cleared before the launch
    unsigned arrive;               // grid barrier: arrivals so far
    unsigned pad0[31];
    unsigned epoch;                // barriers completed, written by the last arrival; polled (a line of its own:
    unsigned abort;                // the polls do not delay the arrivals); a wait expired
    unsigned pad1[30];
    double inertia;
    unsigned long long pad2[15];
};

// Grid-wide barrier number `epoch` (1, 2, ...) for G CTAs.  Returns false when the wait expired or
// another CTA gave up.
__device__ __forceinline__ bool grid_barrier(CoopScratch* sc, unsigned epoch, unsigned G, unsigned spin_limit) {
    __syncthreads();
    __shared__ int s_ok;
    if (threadIdx.x == 0) {
        __threadfence();
        int ok = 0;
        if (atomicAdd(&sc->arrive, 1u) == epoch * G - 1u) {         // the last arrival opens the barrier
            __threadfence();
            *reinterpret_cast<volatile unsigned*>(&sc->epoch) = epoch;
            ok = 1;
        } else {
            for (unsigned i = 0; i < spin_limit; ++i) {
                if (*reinterpret_cast<volatile unsigned*>(&sc->epoch) >= epoch) { ok = 1; break; }
                if ((i & 255u) == 255u && *reinterpret_cast<volatile unsigned*>(&sc->abort)) break;
                __nanosleep(64);
            }
        }
        if (!ok) atomicExch(&sc->abort, 1u);
        __threadfence();
        s_ok = ok;
    }
    __syncthreads();
    return s_ok != 0;
}

// SLOTS threads share the rows of the CTA (a thread owns rows slot and slot + SLOTS); the P = threads / SLOTS
// threads of a slot each scan a contiguous P-th of the centroids, so a CTA with few rows still fills its SM.
template <int D, int SLOTS>
__global__ void __launch_bounds__(cf_threads(D))
fit_coop_kernel(int N, int K, int iters, const float* __restrict__ z, const float* xraw, float* zout,
                const int32_t* __restrict__ init_rows, double* __restrict__ npart /* [G][D][2] column sums per CTA */,
                float* __restrict__ cent,
                int32_t* __restrict__ labels, float* __restrict__ dist2, float* __restrict__ inertia,
                int32_t* __restrict__ rep, int32_t* __restrict__ counts, CoopScratch* __restrict__ sc,
                float* __restrict__ table /* [3][CF_NC][K*D + K] sums then counts (as int) */,
                unsigned long long* __restrict__ rep_key /* [K], cleared */, int* __restrict__ dev_status,
                unsigned spin_limit /* polls of a barrier wait */, int absent_cta /* -1; test only: this CTA never arrives */) {
    kb_grid_dependency_wait();
    if ((int)blockIdx.x == absent_cta) return;                      // (the others give up at their first barrier)
    constexpr int CF_T = cf_threads(D), P = CF_T / SLOTS, CAP = SLOTS * CF_R;
    static_assert(SLOTS % 32 == 0 && P >= 1, "a warp scans one part of the centroids");
    extern __shared__ __align__(16) unsigned char cf_raw[];
    constexpr int ZS = D + 1;                                       // padded row stride: conflict-free column walks
    float* cs = reinterpret_cast<float*>(cf_raw);                   // [K][D] centroids
    float* zs = cs + (size_t)K * D;                                 // [CAP][D+1] this CTA's rows
    float* pbest = zs + (size_t)CAP * ZS;                           // [P][CAP] best distance of each part
    int* parg = reinterpret_cast<int*>(pbest + P * CAP);            // [P][CAP] and its centroid
    float* rbest = reinterpret_cast<float*>(parg + P * CAP);        // [CAP] best over the parts
    int* rarg = reinterpret_cast<int*>(rbest + CAP);                // [CAP]
    int* hist = rarg + CAP;                                         // [K] this CTA's rows per cluster, then the totals
    // [K][D] this CTA's column sums per cluster (16-byte aligned: read as float4)
    float* ssum = reinterpret_cast<float*>((reinterpret_cast<uintptr_t>(hist + K) + 15) & ~(uintptr_t)15);
    __shared__ double s_red[CF_T / 32];
    const int G = gridDim.x, g = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int rows_per = (N + G - 1) / G;
    const int r0 = g * rows_per, rows = max(0, min(N, r0 + rows_per) - r0);      // rows <= CAP (host)
    const int KD = K * D, TS = KD + ((K + 3) & ~3);                 // floats per table (a multiple of four: every copy 16-byte aligned)
    const int slot = tid % SLOTS, part = tid / SLOTS;
    const int kper = (K + P - 1) / P;
    const int jlo = min(K, part * kper), jhi = min(K, jlo + kper);

    // stage this CTA's rows (coalesced float4 reads; plain loads: raw features may be normalised in place)
    // and the initial centroids: the caller's, or the (still raw) rows the caller names
    const unsigned epoch0 = xraw ? 1u : 0u;                         // barriers taken before the Lloyd loop
    const float* zb = (xraw ? xraw : z) + (size_t)r0 * D;
    for (int e = tid; e < rows * (D / 4); e += CF_T) {
        const int r = e / (D / 4), q = e - r * (D / 4);
        const float4 v = *(reinterpret_cast<const float4*>(zb) + e);
        float* d = zs + (size_t)r * ZS + 4 * q;
        d[0] = v.x; d[1] = v.y; d[2] = v.z; d[3] = v.w;
    }
    for (int e = tid; e < KD / 4; e += CF_T) {
        const int j = e / (D / 4), q = e - j * (D / 4);
        const int r = (xraw && init_rows) ? init_rows[j] : -1;
        if (xraw && init_rows && (r < 0 || r >= N)) {
            if (q == 0 && g == 0) atomicOr(dev_status, 4);           // a row id out of range: the centroid stays as it was
        }
        reinterpret_cast<float4*>(cs)[e] = (r >= 0 && r < N) ? *(reinterpret_cast<const float4*>(xraw + (size_t)r * D) + q)
                                                             : __ldg(reinterpret_cast<const float4*>(cent) + e);
    }
    __syncthreads();
    if (xraw) {
        // ---- column z-score over the whole instance (population standard deviation) -------------------
        double* red = reinterpret_cast<double*>(pbest);             // [CF_T][2] (the assign's scratch: free here)
        constexpr int SL = CF_T / D;                                // threads per column
        const int c = tid % D, sl = tid / D;
        const float pivot = xraw[c];                                // first row of the instance: the same shift everywhere
        double s1 = 0.0, s2 = 0.0;
        for (int r = sl; r < rows; r += SL) {
            const float e = zs[(size_t)r * ZS + c] - pivot;
            s1 += (double)e;
            s2 += (double)e * (double)e;
        }
        red[2 * tid] = s1; red[2 * tid + 1] = s2;
        __syncthreads();
        if (tid < D) {
            for (int q = 1; q < SL; ++q) { s1 += red[2 * (q * D + c)]; s2 += red[2 * (q * D + c) + 1]; }
            npart[((size_t)g * D + c) * 2] = s1;
            npart[((size_t)g * D + c) * 2 + 1] = s2;
        }
        if (!grid_barrier(sc, 1u, (unsigned)G, spin_limit)) {
            if (tid == 0) atomicOr(dev_status, CF_STATUS_TIMEOUT);
            return;
        }
        // every CTA adds all partials, slices of the CTA index per thread, then the slices in order
        s1 = 0.0; s2 = 0.0;
        for (int k = sl; k < G; k += SL) {
            s1 += __ldcg(npart + ((size_t)k * D + c) * 2);
            s2 += __ldcg(npart + ((size_t)k * D + c) * 2 + 1);
        }
        red[2 * tid] = s1; red[2 * tid + 1] = s2;
        __syncthreads();
        float* st_mh = reinterpret_cast<float*>(red + 2 * CF_T);    // [D] mean high | [D] mean low | [D] 1 / sd
        if (tid < D) {
            for (int q = 1; q < SL; ++q) { s1 += red[2 * (q * D + c)]; s2 += red[2 * (q * D + c) + 1]; }
            const double ms = s1 / (double)N;
            double var = s2 / (double)N - ms * ms;
            if (var < 0.0) var = 0.0;
            const double mean = (double)pivot + ms;
            const double sd = sqrt(var);
            const double scd = sd < 1e-12 ? 1.0 : sd;               // a constant column is only centred
            const float mh = (float)mean;
            st_mh[c] = mh;
            st_mh[D + c] = (float)(mean - (double)mh);
            st_mh[2 * D + c] = (float)(1.0 / scd);
        }
        __syncthreads();
        float* zo = zout + (size_t)r0 * D;
        for (int e = tid; e < rows * (D / 4); e += CF_T) {
            const int r = e / (D / 4), q = e - r * (D / 4);
            float* d = zs + (size_t)r * ZS + 4 * q;
            float4 v;
            v.x = ((d[0] - st_mh[4 * q]) - st_mh[D + 4 * q]) * st_mh[2 * D + 4 * q];
            v.y = ((d[1] - st_mh[4 * q + 1]) - st_mh[D + 4 * q + 1]) * st_mh[2 * D + 4 * q + 1];
            v.z = ((d[2] - st_mh[4 * q + 2]) - st_mh[D + 4 * q + 2]) * st_mh[2 * D + 4 * q + 2];
            v.w = ((d[3] - st_mh[4 * q + 3]) - st_mh[D + 4 * q + 3]) * st_mh[2 * D + 4 * q + 3];
            d[0] = v.x; d[1] = v.y; d[2] = v.z; d[3] = v.w;
            reinterpret_cast<float4*>(zo)[e] = v;
        }
        if (init_rows)
            for (int e = tid; e < KD; e += CF_T) {
                const int j = e / D, d = e - j * D, r = init_rows[j];
                if (r >= 0 && r < N) cs[e] = ((cs[e] - st_mh[d]) - st_mh[D + d]) * st_mh[2 * D + d];
            }
        __syncthreads();
    }
    float x[CF_R][D];
#pragma unroll
    for (int u = 0; u < CF_R; ++u) {
        const bool active = slot + u * SLOTS < rows;
#pragma unroll
        for (int d = 0; d < D; ++d) x[u][d] = active ? zs[(size_t)(slot + u * SLOTS) * ZS + d] : 0.f;
    }

    bool ok = true;
    for (int it = 0; it <= iters; ++it) {
        // ---- assign: nearest centroid of my rows among my part, then the best over the parts -------------
        {
            float best[CF_R];
            int arg[CF_R];
#pragma unroll
            for (int u = 0; u < CF_R; ++u) { best[u] = INFINITY; arg[u] = 0; }
            for (int j = jlo; j < jhi; ++j) {
                const float4* c4 = reinterpret_cast<const float4*>(cs + (size_t)j * D);
                float acc[CF_R];
#pragma unroll
                for (int u = 0; u < CF_R; ++u) acc[u] = 0.f;
#pragma unroll
                for (int q = 0; q < D / 4; ++q) {
                    const float4 c = c4[q];
#pragma unroll
                    for (int u = 0; u < CF_R; ++u) {
                        const float e0 = x[u][4 * q] - c.x, e1 = x[u][4 * q + 1] - c.y, e2 = x[u][4 * q + 2] - c.z,
                                    e3 = x[u][4 * q + 3] - c.w;
                        acc[u] = fmaf(e0, e0, acc[u]); acc[u] = fmaf(e1, e1, acc[u]);
                        acc[u] = fmaf(e2, e2, acc[u]); acc[u] = fmaf(e3, e3, acc[u]);
                    }
                }
#pragma unroll
                for (int u = 0; u < CF_R; ++u) {
                    if (acc[u] < best[u]) { best[u] = acc[u]; arg[u] = j; }
                }
            }
#pragma unroll
            for (int u = 0; u < CF_R; ++u) {
                pbest[part * CAP + slot + u * SLOTS] = best[u];
                parg[part * CAP + slot + u * SLOTS] = arg[u];
            }
        }
        if (it < iters) {
            for (int e = tid; e < KD; e += CF_T) ssum[e] = 0.f;
            for (int j = tid; j < K; j += CF_T) hist[j] = 0;
        }
        __syncthreads();
        for (int r = tid; r < rows; r += CF_T) {
            float bb = pbest[r];
            int aa = parg[r];
#pragma unroll
            for (int p = 1; p < P; ++p) {                           // parts hold ascending ids: strict < keeps the lowest
                const float v = pbest[p * CAP + r];
                if (v < bb) { bb = v; aa = parg[p * CAP + r]; }
            }
            rbest[r] = bb;
            rarg[r] = aa;
        }
        if (it == iters) break;                                     // the final assign has no update after it

        float* tab0 = table + (size_t)(it % 3) * CF_NC * TS;
        float* tab = tab0 + (size_t)(g % CF_NC) * TS;
        // the first CTAs clear the table of the next iteration (nobody reads or writes it during this one)
        if (g < CF_NC) {
            float* nxt = table + ((size_t)((it + 1) % 3) * CF_NC + g) * TS;
            for (int e = tid; e < TS; e += CF_T) nxt[e] = 0.f;
        }
        // ---- update: (cluster, column) sums of this CTA's rows in shared memory, then into the table ----
        // (ssum and hist were cleared before the combine above)
        __syncthreads();
        for (int e = tid; e < rows * D; e += CF_T) {
            const int r = e / D, d = e - r * D;                     // a warp covers consecutive columns of one row
            const int a = rarg[r];
            atomicAdd(ssum + a * D + d, zs[(size_t)r * ZS + d]);
            if (d == 0) atomicAdd(hist + a, 1);
        }
        __syncthreads();
        for (int e4 = tid; e4 < KD / 4; e4 += CF_T) {               // four columns per reduction: a quarter of the operations
            const int e = 4 * e4, j = e / D, n = hist[j];
            if (n > 0) {
                const float4 v = *reinterpret_cast<const float4*>(ssum + e);
                asm volatile("red.relaxed.gpu.global.add.v4.f32 [%0], {%1, %2, %3, %4};"
                             ::"l"(tab + e), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w) : "memory");
                if (e - j * D == 0) atomicAdd(reinterpret_cast<int*>(tab + KD) + j, n);
            }
        }
        // ---- everybody's sums are in the table after the barrier ---------------------------------
        ok = grid_barrier(sc, epoch0 + (unsigned)(it + 1), (unsigned)G, spin_limit);
        if (!ok) break;
        // written by other CTAs: read through L2; the counts once per cluster (every CTA reads these lines)
        {
            int n[CF_NC];
            const int j = min(tid, K - 1);
#pragma unroll
            for (int c = 0; c < CF_NC; ++c) n[c] = __ldcg(reinterpret_cast<const int*>(tab0 + (size_t)c * TS + KD) + j);
            for (int e0 = 0; e0 < KD; e0 += 4 * CF_T) {
                float v[4][CF_NC];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int e = min(e0 + u * CF_T + tid, KD - 1);
#pragma unroll
                    for (int c = 0; c < CF_NC; ++c) v[u][c] = __ldcg(tab0 + (size_t)c * TS + e);
                }
                if (e0 == 0) {
                    int tot = 0;
#pragma unroll
                    for (int c = 0; c < CF_NC; ++c) tot += n[c];
                    if (tid < K) hist[tid] = tot;
                    for (int jj = tid + CF_T; jj < K; jj += CF_T) {     // K beyond the block: the rest of the counts
                        int t2 = 0;
#pragma unroll
                        for (int c = 0; c < CF_NC; ++c) t2 += __ldcg(reinterpret_cast<const int*>(tab0 + (size_t)c * TS + KD) + jj);
                        hist[jj] = t2;
                    }
                    __syncthreads();
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int e = e0 + u * CF_T + tid;
                    float sum = v[u][0];
#pragma unroll
                    for (int c = 1; c < CF_NC; ++c) sum += v[u][c];
                    const int cnt = e < KD ? hist[e / D] : 0;
                    if (cnt > 0) cs[e] = sum / (float)cnt;          // an empty cluster keeps its centroid
                }
            }
        }
        if (g == 0 && it == iters - 1 && counts)
            for (int j = tid; j < K; j += CF_T) counts[j] = hist[j];
        __syncthreads();
    }
    if (!ok) {
        if (tid == 0) atomicOr(dev_status, CF_STATUS_TIMEOUT);
        return;
    }
    __syncthreads();

    // ---- outputs of the final assign --------------------------------------------------------
    double mine = 0.0;
    for (int lr = tid; lr < rows; lr += CF_T) {
        const int r = r0 + lr, a = rarg[lr];
        const float bb = rbest[lr];
        labels[r] = a;
        if (dist2) dist2[r] = bb;
        mine += (double)bb;
        // the representative is the member with the smallest (dist2, row): keys are stored inverted so
        // that the cleared word means "no member" and atomicMax keeps the smallest key
        if (rep) {                                          // (a key that cannot win is dropped after a cached read)
            const unsigned long long inv = ~(((unsigned long long)__float_as_uint(bb) << 32) | (unsigned)r);
            if (inv > __ldca(rep_key + a)) atomicMax(&rep_key[a], inv);
        }
    }
    if (g == 0) {
        for (int e = tid; e < KD / 4; e += CF_T)
            reinterpret_cast<float4*>(cent)[e] = reinterpret_cast<const float4*>(cs)[e];
        if (iters == 0 && counts)
            for (int j = tid; j < K; j += CF_T) counts[j] = 0;
    }
    if (inertia) {
        const double s = kb_warp_sum(mine);
        if (lane == 0) s_red[warp] = s;
        __syncthreads();
        if (tid == 0) {
            double t = 0.0;
            for (int w = 0; w < CF_T / 32; ++w) t += s_red[w];
            if (t != 0.0) atomicAdd(&sc->inertia, t);
        }
    }
    if (inertia || rep) {
        // one more barrier, then CTA 0 publishes what needed every CTA's contribution
        if (!grid_barrier(sc, epoch0 + (unsigned)(iters + 1), (unsigned)G, spin_limit)) {
            if (tid == 0) atomicOr(dev_status, CF_STATUS_TIMEOUT);
            return;
        }
        if (g == 0) {
            if (inertia && tid == 0) inertia[0] = (float)*reinterpret_cast<volatile double*>(&sc->inertia);
            if (rep)
                for (int j = tid; j < K; j += CF_T) {
                    const unsigned long long inv = __ldcg(rep_key + j);
                    rep[j] = inv == 0ull ? -1 : (int32_t)((~inv) & 0xffffffffull);
                }
        }
    }
}

__global__ void coop_zero_kernel(size_t n16, uint4* __restrict__ p) {
    kb_grid_dependency_wait();
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n16) p[i] = make_uint4(0u, 0u, 0u, 0u);
}

int cf_slots(int rows_per) { return rows_per <= 128 ? 64 : (rows_per <= 256 ? 128 : 256); }
size_t cf_smem(int rows_per, int D, int K) {
    const size_t cap = (size_t)cf_slots(rows_per) * CF_R, P = cf_threads(D) / cf_slots(rows_per);
    // centroids | rows (padded) | per-part best and argument | per-row best and argument | hist | column sums
    return (size_t)K * D * 4 + cap * (D + 1) * 4 + P * cap * 8 + cap * 8 + (size_t)K * 4 + (size_t)K * D * 4 + 64;
}
int cf_ctas(const kb_ctx* ctx, int N) {
    long cap = ((long)N + 63) / 64;                     // at least 64 rows per CTA
    long G = ctx->sm_count < cap ? ctx->sm_count : cap;
    return (int)(G < 1 ? 1 : G);
}
constexpr size_t CF_NPART_BYTES = (size_t)256 * 64 * 2 * 8;   // column sums of up to 256 CTAs x 64 columns (in-kernel normalisation)
size_t cf_tables(int D, int K) { return kb_align256((size_t)3 * CF_NC * (K * D + ((K + 3) & ~3)) * 4); }
size_t cf_scratch(int D, int K) {
    return kb_align256(sizeof(CoopScratch)) + kb_align256((size_t)K * 8) + cf_tables(D, K) + CF_NPART_BYTES + 256;
}

}  // namespace

size_t kb_ws_need_fit_coop(int B, int N, int D, int K) {
    return (B == 1 && (D == 16 || D == 32 || D == 64) && K >= 1 && K <= 1024) ? cf_scratch(D, K) : 0;
}

bool kb_fit_coop_eligible(const kb_ctx* ctx, int B, int N, int D, int K) {
    if (B != 1 || N < 1024 || K < 1 || K > 1024) return false;
    if (D != 16 && D != 32 && D != 64) return false;
    if (!ctx->coop_launch) return false;
    const int G = cf_ctas(ctx, N);
    const int rows_per = (N + G - 1) / G;
    if (rows_per > CF_MAXROWS) return false;
    return cf_smem(rows_per, D, K) + 1024 <= (size_t)ctx->max_smem_optin && ctx->ws_bytes >= cf_scratch(D, K);
}

// z: normalised features (input), or null with xraw (raw features, input), zout (normalised, output; may be xraw
// itself) and init_rows (row ids of the initial centroids; null: `cent` holds them)
kb_status kb_launch_fit_coop(kb_ctx* ctx, int N, int D, int K, int iters, const float* z, const float* xraw, float* zout,
                             const int32_t* init_rows, float* cent, int32_t* labels, float* dist2, float* inertia,
                             int32_t* rep, int32_t* counts) {
    const int G = cf_ctas(ctx, N);
    if (G > 256) return kb_fail(ctx, KB_ERR_UNSUPPORTED, "kb_cluster_fit: more than 256 SMs");
    const int rows_per = (N + G - 1) / G;
    const size_t smem = cf_smem(rows_per, D, K);
    // workspace: barrier words | representative keys | tables.  Cleared here: everything up to the end of
    // the first table (the kernel clears the table of iteration i + 1 during iteration i).
    char* ws = ctx->ws;
    CoopScratch* sc = reinterpret_cast<CoopScratch*>(ws);
    unsigned long long* rep_key = reinterpret_cast<unsigned long long*>(ws + kb_align256(sizeof(CoopScratch)));
    float* table = reinterpret_cast<float*>(reinterpret_cast<char*>(rep_key) + kb_align256((size_t)K * 8));
    double* npart = reinterpret_cast<double*>(reinterpret_cast<char*>(table) + cf_tables(D, K));   // plain stores: never cleared
    const size_t zbytes = (size_t)(reinterpret_cast<char*>(table) - ws) + kb_align256((size_t)CF_NC * (K * D + ((K + 3) & ~3)) * 4);
    kb_launch(coop_zero_kernel, (unsigned)((zbytes / 16 + 255) / 256), 256, 0, ctx->stream, zbytes / 16,
              reinterpret_cast<uint4*>(ws));
    KB_LAUNCH_CHECK(ctx, "coop_zero_kernel");

    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(G);
    cfg.blockDim = dim3(cf_threads(D));
    cfg.dynamicSmemBytes = smem;
    cfg.stream = ctx->stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeCooperative;     // all CTAs resident: they wait on one another
    attr[0].val.cooperative = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e;
#define KB_CF_LAUNCH(DD, SS)                                                                                      \
    do {                                                                                                          \
        KB_SMEM_OPTIN(ctx, (fit_coop_kernel<DD, SS>), smem);                                                      \
        e = cudaLaunchKernelEx(&cfg, fit_coop_kernel<DD, SS>, N, K, iters, z, xraw, zout, init_rows, npart, cent, \
                               labels, dist2, inertia, rep, counts, sc, table, rep_key, ctx->dev_status,         \
                               ctx->dbg_wait_limit ? ctx->dbg_wait_limit : CF_SPIN_LIMIT,                         \
                               ctx->dbg_skip_arrival ? G - 1 : -1);                                               \
    } while (0)
#define KB_CF_LAUNCH_D(DD)                            \
    do {                                              \
        if (slots == 64) KB_CF_LAUNCH(DD, 64);        \
        else if (slots == 128) KB_CF_LAUNCH(DD, 128); \
        else KB_CF_LAUNCH(DD, 256);                   \
    } while (0)
    const int slots = cf_slots(rows_per);
    if (D == 16) KB_CF_LAUNCH_D(16);
    else if (D == 32) KB_CF_LAUNCH_D(32);
    else KB_CF_LAUNCH_D(64);
#undef KB_CF_LAUNCH_D
#undef KB_CF_LAUNCH
    if (e != cudaSuccess) return kb_fail(ctx, KB_ERR_CUDA, "launch of fit_coop_kernel: %s", cudaGetErrorString(e));
    KB_LAUNCH_CHECK(ctx, "fit_coop_kernel");
    return KB_OK;
}
