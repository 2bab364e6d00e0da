// kb_cluster_fit for small instances: one CTA per instance, the whole Lloyd loop in one launch.
//
// When an instance has at most 512 rows and D is 16, 32 or 64, per-call launches dominate
// (a call moves a few KB): iters x (assign, update) + the final assign would be 2*iters+1
// calls of several kernels each.  Here a CTA keeps its instance on chip for all iterations:
//   * a thread owns FF_R rows, kept in registers (FF_R x D floats): every centroid value read
//     from shared memory (a warp-wide float4 broadcast, which costs the shared-memory pipe as
//     much as a full 512-byte access) then feeds FF_R rows, so the loop is bound by its FMAs
//     and not by the broadcasts;
//   * centroids live in shared memory;
//     the distance is the direct form sum (z - c)^2, ascending centroid id, strict <
//     (lowest id on ties) -- the same arithmetic as the row-wise assign kernel;
//   * update: counting sort of the row ids by label in shared memory (integer atomics),
//     then thread (cluster, column) adds up its cluster's rows from a padded shared copy
//     of the instance: no floating-point atomics, bank-conflict free;
//   * the final assign also produces dist2, inertia (double, fixed-order block reduction)
//     and the representative member per cluster (64-bit shared atomicMin on (dist2, row)).
// X is read from HBM exactly once per fit.
//
// The whole-step drivers hand this kernel the RAW features instead (`xraw`): the CTA then also does
// what kb_normalize and kb_init_centroids would have done for its instance -- column statistics of
// the staged rows (shifted by the first row, accumulated in double, threads of a column added in a
// fixed order), z = ((x - mean_hi) - mean_lo) / sd applied in shared memory and written out once,
// initial centroids gathered from the normalised rows -- so a small instance goes from raw
// features to labels in one launch and its features cross HBM once in each direction.
#include "kb_internal.cuh"

namespace {

constexpr int FF_MAXROWS = 512;   // rows per instance at most
// rows per thread (row = tid + u * threads): as many as the register file holds
__host__ __device__ constexpr int ff_rows(int D) { return D <= 32 ? 4 : 2; }

// TOL: the tolerance stop is compiled in (its bookkeeping in the update loop costs the plain loop 13 % otherwise)
template <int D, bool TOL>
__global__ void __launch_bounds__(FF_MAXROWS / ff_rows(D))
fit_fused_kernel(int NCAP, int K, int iters, const float* __restrict__ z, const float* xraw, float* zout,
                 const int32_t* __restrict__ init_rows, float* __restrict__ cent,
                 int32_t* __restrict__ labels, float* __restrict__ dist2, float* __restrict__ inertia,
                 int32_t* __restrict__ rep, int32_t* __restrict__ counts, const int32_t* __restrict__ n_active,
                 const int32_t* __restrict__ run_mask, float tol, int32_t* __restrict__ n_iter,
                 int* __restrict__ dev_status) {
    kb_grid_dependency_wait();
    // An expanding frontier: the instance's arrays have NCAP rows of which the first n_active[b] are candidates
    // (N below); without n_active every row is.  An instance whose run_mask entry is 0 is left exactly as it is.
    if (run_mask && run_mask[blockIdx.x] == 0) return;
    const int N = n_active ? min(max(n_active[blockIdx.x], 0), NCAP) : NCAP;
    constexpr int FF_R = ff_rows(D), FF_T = FF_MAXROWS / FF_R;
    extern __shared__ __align__(16) unsigned char ff_raw[];
    constexpr int ZS = D + 1;                                       // padded row stride: conflict-free column walks
    float* cs = reinterpret_cast<float*>(ff_raw);                   // [K][D] centroids (16-byte aligned rows)
    float* zs = cs + (size_t)K * D;                                 // [N][D+1] the instance
    // [K] counts, then scatter cursors; 8-byte aligned because the space is reused for 64-bit keys
    int* hist = reinterpret_cast<int*>((reinterpret_cast<uintptr_t>(zs + (size_t)NCAP * ZS) + 7) & ~(uintptr_t)7);
    int* offs = hist + K;                                           // [K+1]
    unsigned short* perm = reinterpret_cast<unsigned short*>(offs + K + 1);   // [NCAP] row ids in label order
    __shared__ double s_red[FF_MAXROWS / 64];
    __shared__ int s_scan[FF_MAXROWS / 64];
    const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const float* zb = (xraw ? xraw : z) + (size_t)b * NCAP * D;
    float* cb = cent + (size_t)b * K * D;
    if (N == 0) {                                                   // nothing to cluster: centroids stay, every cluster is empty
        for (int j = tid; j < K; j += FF_T) {
            if (counts) counts[(size_t)b * K + j] = 0;
            if (rep) rep[(size_t)b * K + j] = -1;
        }
        if (inertia && tid == 0) inertia[b] = 0.f;
        if (n_iter && tid == 0) n_iter[b] = 0;
        return;
    }

    // stage the instance (coalesced float4 reads; plain loads: raw features may be normalised in place)
    for (int e = tid; e < N * (D / 4); e += FF_T) {
        const int r = e / (D / 4), q = e - r * (D / 4);
        const float4 v = *(reinterpret_cast<const float4*>(zb) + e);
        float* d = zs + (size_t)r * ZS + 4 * q;
        d[0] = v.x; d[1] = v.y; d[2] = v.z; d[3] = v.w;
    }
    __syncthreads();
    if (xraw) {
        // ---- column z-score of the staged rows (population standard deviation) ----------------
        double* red = reinterpret_cast<double*>((reinterpret_cast<uintptr_t>(perm + NCAP) + 7) & ~(uintptr_t)7);   // [FF_T][2]
        float* st_mh = reinterpret_cast<float*>(red + 2 * FF_T);    // [D] mean, high part
        float* st_ml = st_mh + D;                                   // [D] mean, low part
        float* st_inv = st_ml + D;                                  // [D] 1 / standard deviation
        constexpr int SL = FF_T / D;                                // threads per column
        const int c = tid % D, sl = tid / D;
        const float pivot = zs[c];                                  // first row: the same shift for every thread
        double s1 = 0.0, s2 = 0.0;
        for (int r = sl; r < N; r += SL) {
            const float e = zs[(size_t)r * ZS + c] - pivot;
            s1 += (double)e;
            s2 += (double)e * (double)e;
        }
        red[2 * tid] = s1; red[2 * tid + 1] = s2;
        __syncthreads();
        if (tid < D) {
            for (int q = 1; q < SL; ++q) { s1 += red[2 * (q * D + c)]; s2 += red[2 * (q * D + c) + 1]; }
            const double ms = s1 / (double)N;
            double var = s2 / (double)N - ms * ms;
            if (var < 0.0) var = 0.0;
            const double mean = (double)pivot + ms;
            const double sd = sqrt(var);
            const double sc = sd < 1e-12 ? 1.0 : sd;                // a constant column is only centred
            const float mh = (float)mean;
            st_mh[c] = mh;
            st_ml[c] = (float)(mean - (double)mh);
            st_inv[c] = (float)(1.0 / sc);
        }
        __syncthreads();
        float* zo = zout + (size_t)b * NCAP * D;
        for (int e = tid; e < N * (D / 4); e += FF_T) {
            const int r = e / (D / 4), q = e - r * (D / 4);
            float* d = zs + (size_t)r * ZS + 4 * q;
            float4 v;
            v.x = ((d[0] - st_mh[4 * q]) - st_ml[4 * q]) * st_inv[4 * q];
            v.y = ((d[1] - st_mh[4 * q + 1]) - st_ml[4 * q + 1]) * st_inv[4 * q + 1];
            v.z = ((d[2] - st_mh[4 * q + 2]) - st_ml[4 * q + 2]) * st_inv[4 * q + 2];
            v.w = ((d[3] - st_mh[4 * q + 3]) - st_ml[4 * q + 3]) * st_inv[4 * q + 3];
            d[0] = v.x; d[1] = v.y; d[2] = v.z; d[3] = v.w;
            reinterpret_cast<float4*>(zo)[e] = v;
        }
        __syncthreads();
    }
    // initial centroids: the caller's, or the normalised rows the caller names
    for (int e = tid; e < K * D / 4; e += FF_T) {
        float4 v;
        const int j = e / (D / 4), q = e - j * (D / 4);
        const int r = init_rows ? init_rows[(size_t)b * K + j] : -2;
        if (init_rows && r >= 0 && r < N) {
            const float* d = zs + (size_t)r * ZS + 4 * q;
            v = make_float4(d[0], d[1], d[2], d[3]);
        } else if (r == -1) {
            v = make_float4(KB_UNUSED_CENTROID, KB_UNUSED_CENTROID, KB_UNUSED_CENTROID, KB_UNUSED_CENTROID);   // an unused cluster
        } else {
            if (init_rows && q == 0) atomicOr(dev_status, 4);        // a row id out of range: the centroid stays as it was
            v = *(reinterpret_cast<const float4*>(cb) + e);
        }
        reinterpret_cast<float4*>(cs)[e] = v;
    }
    __syncthreads();
    bool active[FF_R];
    float x[FF_R][D];
#pragma unroll
    for (int u = 0; u < FF_R; ++u) {
        active[u] = tid + u * FF_T < N;
#pragma unroll
        for (int d = 0; d < D; ++d) x[u][d] = active[u] ? zs[(size_t)(tid + u * FF_T) * ZS + d] : 0.f;
    }

    float best[FF_R];
    int arg[FF_R];
    int done_updates = 0;
    for (int it = 0; it <= iters; ++it) {
        // ---- assign: nearest centroid of my rows ------------------------------------------
#pragma unroll
        for (int u = 0; u < FF_R; ++u) { best[u] = INFINITY; arg[u] = 0; }
        for (int j = 0; j < K; ++j) {
            const float4* c4 = reinterpret_cast<const float4*>(cs + (size_t)j * D);
            float acc[FF_R];
#pragma unroll
            for (int u = 0; u < FF_R; ++u) acc[u] = 0.f;
#pragma unroll
            for (int q = 0; q < D / 4; ++q) {
                const float4 c = c4[q];
#pragma unroll
                for (int u = 0; u < FF_R; ++u) {
                    const float e0 = x[u][4 * q] - c.x, e1 = x[u][4 * q + 1] - c.y, e2 = x[u][4 * q + 2] - c.z,
                                e3 = x[u][4 * q + 3] - c.w;
                    acc[u] = fmaf(e0, e0, acc[u]); acc[u] = fmaf(e1, e1, acc[u]);
                    acc[u] = fmaf(e2, e2, acc[u]); acc[u] = fmaf(e3, e3, acc[u]);
                }
            }
#pragma unroll
            for (int u = 0; u < FF_R; ++u)
                if (acc[u] < best[u]) { best[u] = acc[u]; arg[u] = j; }
        }
        if (it == iters) break;                                     // the final assign has no update after it
        // ---- update: counting sort by label, then (cluster, column) sums ----------------------
        for (int j = tid; j < K; j += FF_T) hist[j] = 0;
        __syncthreads();
#pragma unroll
        for (int u = 0; u < FF_R; ++u)
            if (active[u]) atomicAdd(&hist[arg[u]], 1);
        __syncthreads();
        {   // exclusive scan of hist (K may exceed the block: contiguous slices per thread)
            const int per = (K + FF_T - 1) / FF_T;
            const int j0 = min(K, tid * per), j1 = min(K, j0 + per);
            int local = 0;
            for (int j = j0; j < j1; ++j) local += hist[j];
            int incl = local;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int v = __shfl_up_sync(0xffffffffu, incl, o);
                if (lane >= o) incl += v;
            }
            if (lane == 31) s_scan[warp] = incl;
            __syncthreads();
            int base = 0;
            for (int w = 0; w < warp; ++w) base += s_scan[w];
            int run = base + incl - local;
            for (int j = j0; j < j1; ++j) { offs[j] = run; run += hist[j]; }
            if (tid == FF_T - 1) offs[K] = run;
        }
        __syncthreads();
        for (int j = tid; j < K; j += FF_T) hist[j] = offs[j];      // scatter cursors
        __syncthreads();
#pragma unroll
        for (int u = 0; u < FF_R; ++u)
            if (active[u]) perm[atomicAdd(&hist[arg[u]], 1)] = (unsigned short)(tid + u * FF_T);
        __syncthreads();
        if ((it == iters - 1 || TOL) && counts)                     // (with a tolerance stop any update may be the last)
            for (int j = tid; j < K; j += FF_T) counts[(size_t)b * K + j] = offs[j + 1] - offs[j];
        float moved = 0.f;                                          // my share of sum_j ||c_j(new) - c_j(old)||^2 (TOL only)
        for (int e = tid; e < K * D; e += FF_T) {
            const int j = e / D, d = e - j * D;                     // a warp covers consecutive columns of one cluster
            const int p0 = offs[j], p1 = offs[j + 1];
            if (p1 > p0) {                                          // an empty cluster keeps its centroid
                float s0 = 0.f, s1 = 0.f;
                int p = p0;
                for (; p + 1 < p1; p += 2) {
                    s0 += zs[(size_t)perm[p] * ZS + d];
                    s1 += zs[(size_t)perm[p + 1] * ZS + d];
                }
                if (p < p1) s0 += zs[(size_t)perm[p] * ZS + d];
                const float c_new = (s0 + s1) / (float)(p1 - p0);
                if (TOL) { const float dlt = c_new - cs[e]; moved = fmaf(dlt, dlt, moved); }
                cs[e] = c_new;
            }
        }
        ++done_updates;
        if (TOL) {
            // tolerance stop: the whole CTA agrees on the instance's total shift (fixed-order block sum)
            const double w = kb_warp_sum((double)moved);
            if (lane == 0) s_red[warp] = w;
            __syncthreads();
            double shift = 0.0;
            for (int q = 0; q < FF_T / 32; ++q) shift += s_red[q];
            if (shift <= (double)tol) iters = it + 1;               // this update stays; the next pass is the final assign
        }
        __syncthreads();
    }
    if (n_iter && tid == 0) n_iter[b] = done_updates;

    // ---- outputs of the final assign --------------------------------------------------------
    unsigned long long* rep_key = reinterpret_cast<unsigned long long*>(hist);   // hist/offs are free now: [K] keys
    if (rep) {
        __syncthreads();
        for (int j = tid; j < K; j += FF_T) rep_key[j] = ~0ull;
        __syncthreads();
    }
#pragma unroll
    for (int u = 0; u < FF_R; ++u)
        if (active[u]) {
            const int r = tid + u * FF_T;
            const size_t flat = (size_t)b * NCAP + r;
            labels[flat] = arg[u];
            if (dist2) dist2[flat] = best[u];
            if (rep) atomicMin(&rep_key[arg[u]], ((unsigned long long)__float_as_uint(best[u]) << 32) | (unsigned)r);
        }
    for (int e = tid; e < K * D / 4; e += FF_T)
        reinterpret_cast<float4*>(cb)[e] = reinterpret_cast<const float4*>(cs)[e];
    if (iters == 0 && counts)
        for (int j = tid; j < K; j += FF_T) counts[(size_t)b * K + j] = 0;
    if (inertia) {
        double mine = 0.0;
#pragma unroll
        for (int u = 0; u < FF_R; ++u) mine += active[u] ? (double)best[u] : 0.0;
        double s = kb_warp_sum(mine);
        if (lane == 0) s_red[warp] = s;
    }
    __syncthreads();
    if (inertia && tid == 0) {
        double s = 0.0;
        for (int w = 0; w < FF_T / 32; ++w) s += s_red[w];
        inertia[b] = (float)s;
    }
    if (rep)
        for (int j = tid; j < K; j += FF_T) {
            const unsigned long long key = rep_key[j];
            rep[(size_t)b * K + j] = key == ~0ull ? -1 : (int32_t)(key & 0xffffffffull);
        }
}

size_t ff_smem(int N, int D, int K) {
    // centroids | instance (padded) | hist [K] + offs [K+1] (reused as K 64-bit keys: needs 2K ints) | perm
    // ... | column statistics of the in-kernel normalisation: [threads][2] doubles and three floats per column
    return (size_t)K * D * 4 + (size_t)N * (D + 1) * 4 + 8 + (size_t)(2 * K + 2) * 4 + (size_t)N * 2 + 16 +
           8 + (size_t)(FF_MAXROWS / 2) * 16 + 3 * 64 * 4;
}

}  // namespace

bool kb_fit_fused_eligible(const kb_ctx* ctx, int B, int N, int D, int K) {
    if (B < 1 || N < 1 || N > FF_MAXROWS || K < 1 || K > 4096) return false;
    if (D != 16 && D != 32 && D != 64) return false;
    return ff_smem(N, D, K) + 256 <= (size_t)ctx->max_smem_optin;
}

// z: normalised features (input), or null with xraw (raw features, input), zout (normalised, output; may be
// xraw itself) and init_rows (row ids of the initial centroids; null: `cent` holds them)
kb_status kb_launch_fit_fused(kb_ctx* ctx, int B, int N, int D, int K, int iters, const float* z, const float* xraw,
                              float* zout, const int32_t* init_rows, float* cent, int32_t* labels, float* dist2,
                              float* inertia, int32_t* rep, int32_t* counts, const int32_t* n_active,
                              const int32_t* run_mask, float tol, int32_t* n_iter) {
    const size_t smem = ff_smem(N, D, K);
#define KB_FF_LAUNCH(DD, TT)                                                                                             \
    do {                                                                                                                 \
        KB_SMEM_OPTIN(ctx, (fit_fused_kernel<DD, TT>), smem);                                                            \
        kb_launch(fit_fused_kernel<DD, TT>, B, FF_MAXROWS / ff_rows(DD), smem, ctx->stream, N, K, iters, z, xraw, zout,  \
                  init_rows, cent, labels, dist2, inertia, rep, counts, n_active, run_mask, tol, n_iter, ctx->dev_status); \
    } while (0)
    const bool stop = tol >= 0.f;
    if (D == 16) { if (stop) KB_FF_LAUNCH(16, true); else KB_FF_LAUNCH(16, false); }
    else if (D == 32) { if (stop) KB_FF_LAUNCH(32, true); else KB_FF_LAUNCH(32, false); }
    else { if (stop) KB_FF_LAUNCH(64, true); else KB_FF_LAUNCH(64, false); }
#undef KB_FF_LAUNCH
    KB_LAUNCH_CHECK(ctx, "fit_fused_kernel");
    return KB_OK;
}
