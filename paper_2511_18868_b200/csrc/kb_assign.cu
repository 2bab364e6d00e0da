// kb_cluster_assign: nearest centroid in squared Euclidean distance (K-Means
// assignment, Sec. 3.3).
//
// Row-wise fp32 FFMA path: one thread owns one row (kept in shared memory with
// an odd row stride, so the 32 rows of a warp sit in 32 different banks), the
// centroids stream through shared memory in groups of eight and are read as
// warp-wide broadcasts.  The distance is the direct form sum (z - c)^2, so the
// reported dist2 carries no cancellation error.  Optional outputs: inertia
// (double atomics, one per block) and the representative member per cluster
// (64-bit atomicMin on the pair (dist2 bits, k): lowest k wins a tie).
#include "kb_internal.cuh"

namespace {

constexpr int AS_GROUP = 8;  // centroids evaluated per pass over a row

// layout of the assign scratch: inertia double[B] | rep uint64[B][K]
__global__ void assign_finalize_kernel(int B, int K, const double* __restrict__ ws_inertia,
                                       const unsigned long long* __restrict__ ws_rep, float* __restrict__ inertia,
                                       int32_t* __restrict__ rep) {
    kb_grid_dependency_wait();
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (inertia && i < B) inertia[i] = (float)ws_inertia[i];
    if (rep && i < B * K) {
        unsigned long long key = ws_rep[i];
        rep[i] = key == ~0ull ? -1 : (int32_t)(key & 0xffffffffull);
    }
}

template <bool VEC4>
__global__ void __launch_bounds__(128)
assign_rowwise_kernel(int N, int D, int K, int TM, int CT, const float* __restrict__ z,
                      const float* __restrict__ cent, int32_t* __restrict__ labels, float* __restrict__ dist2,
                      double* __restrict__ ws_inertia, unsigned long long* __restrict__ ws_rep) {
    kb_grid_dependency_wait();
    extern __shared__ __align__(16) float smem[];
    const int XS = D + 1;                    // odd stride when D is even; any stride is correct
    float* cs = smem;                        // [CT][D]     (16-byte aligned rows when D % 4 == 0)
    float* xs = smem + (size_t)CT * D;       // [TM][XS]
    const int b = blockIdx.y, tid = threadIdx.x;
    const int r0 = blockIdx.x * TM;
    const int rows = min(TM, N - r0);
    const float* zb = z + ((size_t)b * N + r0) * D;
    const float* cb = cent + (size_t)b * K * D;

    // stage the row tile (coalesced reads, scalar stores into the padded tile)
    if (VEC4) {
        const int vpr = D >> 2;
        for (int e = tid; e < rows * vpr; e += blockDim.x) {
            int r = e / vpr, q = e - r * vpr;
            float4 v = __ldg(reinterpret_cast<const float4*>(zb + (size_t)r * D) + q);
            float* d = xs + (size_t)r * XS + 4 * q;
            d[0] = v.x; d[1] = v.y; d[2] = v.z; d[3] = v.w;
        }
    } else {
        for (int e = tid; e < rows * D; e += blockDim.x) {
            int r = e / D, d = e - r * D;
            xs[(size_t)r * XS + d] = __ldg(zb + e);
        }
    }

    float best = INFINITY;
    int arg = 0;
    const bool active = tid < rows;
    const float* xr = xs + (size_t)(active ? tid : 0) * XS;

    for (int j0 = 0; j0 < K; j0 += CT) {
        const int nc = min(CT, K - j0);
        __syncthreads();  // previous tile consumed (and, first time, the row tile is complete)
        if (VEC4) {
            const float4* src = reinterpret_cast<const float4*>(cb + (size_t)j0 * D);
            float4* dst = reinterpret_cast<float4*>(cs);
            for (int e = tid; e < (nc * D) >> 2; e += blockDim.x) dst[e] = __ldg(src + e);
        } else {
            for (int e = tid; e < nc * D; e += blockDim.x) cs[e] = __ldg(cb + (size_t)j0 * D + e);
        }
        __syncthreads();
        if (!active) continue;
        for (int g0 = 0; g0 < nc; g0 += AS_GROUP) {
            float acc[AS_GROUP];
#pragma unroll
            for (int u = 0; u < AS_GROUP; ++u) acc[u] = 0.f;
            // rows past the end of the tile are clamped to the last one and ignored below
            const float* c0 = cs + (size_t)g0 * D;
            int off[AS_GROUP];
#pragma unroll
            for (int u = 0; u < AS_GROUP; ++u) off[u] = min(u, nc - 1 - g0) * D;
            if (VEC4) {
                for (int d = 0; d < D; d += 4) {
                    float x0 = xr[d], x1 = xr[d + 1], x2 = xr[d + 2], x3 = xr[d + 3];
#pragma unroll
                    for (int u = 0; u < AS_GROUP; ++u) {
                        float4 c = *reinterpret_cast<const float4*>(c0 + off[u] + d);
                        float e0 = x0 - c.x, e1 = x1 - c.y, e2 = x2 - c.z, e3 = x3 - c.w;
                        acc[u] = fmaf(e0, e0, acc[u]);
                        acc[u] = fmaf(e1, e1, acc[u]);
                        acc[u] = fmaf(e2, e2, acc[u]);
                        acc[u] = fmaf(e3, e3, acc[u]);
                    }
                }
            } else {
                for (int d = 0; d < D; ++d) {
                    float x0 = xr[d];
#pragma unroll
                    for (int u = 0; u < AS_GROUP; ++u) {
                        float e0 = x0 - c0[off[u] + d];
                        acc[u] = fmaf(e0, e0, acc[u]);
                    }
                }
            }
#pragma unroll
            for (int u = 0; u < AS_GROUP; ++u)
                if (g0 + u < nc && acc[u] < best) { best = acc[u]; arg = j0 + g0 + u; }
        }
    }

    if (active) {
        const size_t i = (size_t)b * N + r0 + tid;
        labels[i] = arg;
        if (dist2) dist2[i] = best;
        if (ws_rep) {
            // all rows of a cluster meet in one word: only a key that beats the value seen so far (a cached,
            // possibly stale, hence larger one) goes to the atomic unit
            const unsigned long long key = ((unsigned long long)__float_as_uint(best) << 32) | (unsigned)(r0 + tid);
            unsigned long long* slot = &ws_rep[(size_t)b * K + arg];
            if (key < __ldca(slot)) atomicMin(slot, key);
        }
    }
    if (ws_inertia) {
        double s = kb_warp_sum(active ? (double)best : 0.0);
        if ((tid & 31) == 0 && s != 0.0) atomicAdd(&ws_inertia[b], s);
    }
}

}  // namespace

size_t kb_ws_need_assign(int B, int N, int D, int K) {
    // generic scratch (inertia double[B] | rep uint64[B][K]) followed by the tensor path's scratch
    return kb_align256((size_t)B * sizeof(double)) + kb_align256((size_t)B * K * sizeof(unsigned long long)) +
           kb_ws_need_assign_tc(B, N, D, K);
}

static kb_status launch_rowwise(kb_ctx* ctx, int B, int N, int D, int K, const float* z, const float* c,
                                int32_t* labels, float* dist2, double* ws_inertia, unsigned long long* ws_rep) {
    // rows per block: as many as fit beside the centroid tile in 96 KB, at most 128
    const size_t budget = 96 * 1024;
    int CT = (int)((16 * 1024) / ((size_t)D * 4));
    CT = CT / AS_GROUP * AS_GROUP;
    if (CT < AS_GROUP) CT = AS_GROUP;
    if (CT > ((K + AS_GROUP - 1) / AS_GROUP) * AS_GROUP) CT = ((K + AS_GROUP - 1) / AS_GROUP) * AS_GROUP;
    size_t cbytes = (size_t)CT * D * 4;
    if (cbytes + (size_t)32 * (D + 1) * 4 > budget)
        return kb_fail(ctx, KB_ERR_UNSUPPORTED, "kb_cluster_assign: D = %d is beyond the row-wise path", D);
    int TM = (int)((budget - cbytes) / ((size_t)(D + 1) * 4));
    TM = TM >= 128 ? 128 : (TM / 32 * 32);
    size_t smem = cbytes + (size_t)TM * (D + 1) * 4;
    dim3 grid((N + TM - 1) / TM, B);
    if (D % 4 == 0) {
        KB_SMEM_OPTIN(ctx, assign_rowwise_kernel<true>, smem);
        kb_launch(assign_rowwise_kernel<true>, grid, 128, smem, ctx->stream, N, D, K, TM, CT, z, c, labels, dist2,
                                                                     ws_inertia, ws_rep);
    } else {
        KB_SMEM_OPTIN(ctx, assign_rowwise_kernel<false>, smem);
        kb_launch(assign_rowwise_kernel<false>, grid, 128, smem, ctx->stream, N, D, K, TM, CT, z, c, labels, dist2,
                                                                      ws_inertia, ws_rep);
    }
    KB_LAUNCH_CHECK(ctx, "assign_rowwise_kernel");
    return KB_OK;
}

kb_status kb_launch_assign(kb_ctx* ctx, int B, int N, int D, int K, const float* z, const float* c, int32_t* labels,
                           float* dist2, float* inertia, int32_t* rep) {
    if (B == 0) return KB_OK;
    const bool use_tc = N > 0 && ctx->assign_path != 1 &&
                        (ctx->assign_path >= 2 ? kb_assign_tc_supported(ctx, B, D, K) : kb_assign_tc_eligible(ctx, B, N, D, K));
    if (ctx->assign_path >= 2 && N > 0 && !use_tc)
        return kb_fail(ctx, KB_ERR_UNSUPPORTED, "kb_cluster_assign: the tensor path needs D %% 32 == 0, D <= 128");
    double* ws_inertia = nullptr;
    unsigned long long* ws_rep = nullptr;
    const size_t off_rep = kb_align256((size_t)B * sizeof(double));
    const size_t off_tc = off_rep + kb_align256((size_t)B * K * sizeof(unsigned long long));
    if (inertia || rep || use_tc) {
        const size_t need = use_tc ? kb_ws_need_assign(B, N, D, K) : off_tc;
        if (ctx->ws_bytes < need)
            return kb_fail(ctx, KB_ERR_WORKSPACE, "kb_cluster_assign needs %zu bytes of workspace", need);
    }
    if (inertia) {
        ws_inertia = reinterpret_cast<double*>(ctx->ws);
        KB_MEMSET(ctx, ws_inertia, 0, (size_t)B * sizeof(double));
    }
    if (rep) {
        ws_rep = reinterpret_cast<unsigned long long*>(ctx->ws + off_rep);
        KB_MEMSET(ctx, ws_rep, 0xff, (size_t)B * K * sizeof(unsigned long long));
    }
    ctx->last_assign_path = 0;
    if (N > 0) {
        kb_status s;
        if (use_tc) {
            s = kb_launch_assign_tc(ctx, ctx->ws + off_tc, B, N, D, K, z, c, labels, nullptr, nullptr, ctx->tc_eps);
            if (s == KB_OK && (dist2 || inertia || rep))
                s = kb_launch_assign_finish(ctx, B, N, D, K, z, c, labels, dist2, ws_inertia, ws_rep);
            ctx->last_assign_path = ctx->assign_path == 3 ? 3 : 2;
        } else {
            s = launch_rowwise(ctx, B, N, D, K, z, c, labels, dist2, ws_inertia, ws_rep);
            ctx->last_assign_path = 1;
            ctx->last_assign_presplit = 0;
        }
        if (s != KB_OK) return s;
    }
    if (inertia || rep) {
        int total = B * (rep ? K : 1);
        kb_launch(assign_finalize_kernel, (total + 255) / 256, 256, 0, ctx->stream, B, K, ws_inertia, ws_rep, inertia, rep);
        KB_LAUNCH_CHECK(ctx, "assign_finalize_kernel");
    }
    return KB_OK;
}
