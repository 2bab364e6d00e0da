// kb_normalize: per instance and column population z-score (feature
// normalisation of Sec. 3.2 / App. A.1).
//
// Two streaming passes over X: (1) per-block shifted sums (fp32 runs of eight, widened to
// double), then a small kernel that adds the per-block partials of every column in a fixed
// order; (2) apply.  HBM traffic is read + read + write = 12 bytes per element (8 when X stays
// in L2 between the passes).
#include "kb_internal.cuh"

namespace {

template <int V> struct Vec;
template <> struct Vec<4> { typedef float4 type; };
template <> struct Vec<1> { typedef float type; };

template <int V> __device__ __forceinline__ void ld(const float* p, float (&v)[V]);
template <> __device__ __forceinline__ void ld<4>(const float* p, float (&v)[4]) {
    float4 t = __ldg(reinterpret_cast<const float4*>(p));
    v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
}
template <> __device__ __forceinline__ void ld<1>(const float* p, float (&v)[1]) { v[0] = __ldg(p); }
// plain (coherent) load: the apply pass may run in place
template <int V> __device__ __forceinline__ void ldp(const float* p, float (&v)[V]);
template <> __device__ __forceinline__ void ldp<4>(const float* p, float (&v)[4]) {
    float4 t = *reinterpret_cast<const float4*>(p);
    v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
}
template <> __device__ __forceinline__ void ldp<1>(const float* p, float (&v)[1]) { v[0] = *p; }
template <int V> __device__ __forceinline__ void st(float* p, const float (&v)[V]);
template <> __device__ __forceinline__ void st<4>(float* p, const float (&v)[4]) {
    *reinterpret_cast<float4*>(p) = make_float4(v[0], v[1], v[2], v[3]);
}
template <> __device__ __forceinline__ void st<1>(float* p, const float (&v)[1]) { *p = v[0]; }

// Thread geometry shared by both passes: a block covers CW column-vectors
// (one "chunk" of the row) x RL row lanes; blockIdx.y selects the chunk.
struct Geo {
    int cpr;  // column vectors per row (D / V)
    int cw;   // column vectors per chunk (<= 256)
    int rl;   // row lanes per block
};

template <int V>
__global__ void __launch_bounds__(256)
norm_stats_kernel(int N, int D, Geo g, int G, const float* __restrict__ x, double* __restrict__ part) {
    kb_grid_dependency_wait();
    extern __shared__ double red[];  // [threads][2V]
    const int b = blockIdx.z, chunk = blockIdx.y, blk = blockIdx.x;
    const int tid = threadIdx.x, T = g.cw * g.rl;
    const int cl = tid % g.cw, rl = tid / g.cw;
    const int cq = chunk * g.cw + cl;
    const bool active = tid < T && cq < g.cpr;
    const float* xb = x + (size_t)b * N * D;
    const int rows_per = (N + G - 1) / G;
    const int r0 = blk * rows_per, r1 = min(N, r0 + rows_per);

    double s1[V], s2[V];
#pragma unroll
    for (int i = 0; i < V; ++i) { s1[i] = 0.0; s2[i] = 0.0; }
    if (active) {
        float shift[V];
        ld<V>(xb + (size_t)cq * V, shift);  // first row of the instance: same pivot in every block
        for (int rb = r0 + rl; rb < r1; rb += 8 * g.rl) {
            // eight independent loads in flight, a short fp32 run over them, then widen
            float v[8][V];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int r = rb + u * g.rl;
                if (r < r1) {
                    ld<V>(xb + (size_t)r * D + (size_t)cq * V, v[u]);
                } else {
#pragma unroll
                    for (int i = 0; i < V; ++i) v[u][i] = shift[i];   // contributes exactly zero
                }
            }
            float f1[V], f2[V];
#pragma unroll
            for (int i = 0; i < V; ++i) { f1[i] = 0.f; f2[i] = 0.f; }
#pragma unroll
            for (int u = 0; u < 8; ++u) {
#pragma unroll
                for (int i = 0; i < V; ++i) {
                    float e = v[u][i] - shift[i];
                    f1[i] += e;
                    f2[i] = fmaf(e, e, f2[i]);
                }
            }
#pragma unroll
            for (int i = 0; i < V; ++i) { s1[i] += (double)f1[i]; s2[i] += (double)f2[i]; }
        }
    }
    // block reduction over the row lanes, in a fixed order
#pragma unroll
    for (int i = 0; i < V; ++i) { red[(size_t)tid * 2 * V + i] = s1[i]; red[(size_t)tid * 2 * V + V + i] = s2[i]; }
    __syncthreads();
    if (active && rl == 0) {
        for (int q = 1; q < g.rl; ++q) {
            const double* o = red + (size_t)(q * g.cw + cl) * 2 * V;
#pragma unroll
            for (int i = 0; i < V; ++i) { s1[i] += o[i]; s2[i] += o[V + i]; }
        }
        double* dst = part + (((size_t)b * G + blk) * D + (size_t)cq * V) * 2;
#pragma unroll
        for (int i = 0; i < V; ++i) { dst[2 * i] = s1[i]; dst[2 * i + 1] = s2[i]; }
    }
}

// Adds the per-block partials of each column in a fixed order and derives the statistics.
// A block takes NC_COLS columns of one instance; NC_SL threads per column each add a contiguous
// slice of the partial index (eight loads in flight), the slices are then added in order.
constexpr int NC_COLS = 4, NC_SL = 64;
__global__ void __launch_bounds__(NC_COLS * NC_SL)
norm_combine_kernel(int N, int D, int G, const float* __restrict__ x, const double* __restrict__ part,
                    float* __restrict__ stat, float* __restrict__ mean_out, float* __restrict__ scale_out) {
    kb_grid_dependency_wait();
    __shared__ double s_a[NC_SL][NC_COLS], s_q[NC_SL][NC_COLS];
    const int b = blockIdx.y, tid = threadIdx.x;
    const int cc = tid % NC_COLS, sl = tid / NC_COLS;
    const int col = blockIdx.x * NC_COLS + cc;
    const int per = (G + NC_SL - 1) / NC_SL;
    double a = 0.0, q = 0.0;
    if (col < D) {
        const int k1 = min(G, (sl + 1) * per);
        const size_t st = (size_t)D * 2;
        int k = sl * per;
        for (; k + 7 < k1; k += 8) {
            const double* p0 = part + (((size_t)b * G + k) * D + col) * 2;
            double va[8], vq[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) { va[u] = p0[u * st]; vq[u] = p0[u * st + 1]; }
#pragma unroll
            for (int u = 0; u < 8; ++u) { a += va[u]; q += vq[u]; }
        }
        for (; k < k1; ++k) {
            const double* p = part + (((size_t)b * G + k) * D + col) * 2;
            a += p[0];
            q += p[1];
        }
    }
    s_a[sl][cc] = a; s_q[sl][cc] = q;
    __syncthreads();
    if (sl != 0 || col >= D) return;
    for (int k = 1; k < NC_SL; ++k) { a += s_a[k][cc]; q += s_q[k][cc]; }
    const float* xb = x + (size_t)b * N * D;
    double ms = a / (double)N;
    double var = q / (double)N - ms * ms;
    if (var < 0.0) var = 0.0;
    double mean = (double)__ldg(xb + col) + ms;
    double sd = sqrt(var);
    double sc = sd < 1e-12 ? 1.0 : sd;
    float mh = (float)mean;
    float* sp = stat + ((size_t)b * D + col) * 4;
    sp[0] = mh;
    sp[1] = (float)(mean - (double)mh);
    sp[2] = (float)(1.0 / sc);
    sp[3] = (float)sc;
    if (mean_out) mean_out[(size_t)b * D + col] = mh;
    if (scale_out) scale_out[(size_t)b * D + col] = (float)sc;
}

template <int V>
__global__ void __launch_bounds__(256)
norm_apply_kernel(int N, int D, Geo g, int G, const float* x, float* z, const float* __restrict__ stat) {
    kb_grid_dependency_wait();
    const int b = blockIdx.z, chunk = blockIdx.y, blk = blockIdx.x;
    const int tid = threadIdx.x, T = g.cw * g.rl;
    const int cl = tid % g.cw, rl = tid / g.cw;
    const int cq = chunk * g.cw + cl;
    if (tid >= T || cq >= g.cpr) return;
    const float* xb = x + (size_t)b * N * D;
    float* zb = z + (size_t)b * N * D;
    const int rows_per = (N + G - 1) / G;
    const int r0 = blk * rows_per, r1 = min(N, r0 + rows_per);
    float mh[V], ml[V], inv[V];
#pragma unroll
    for (int i = 0; i < V; ++i) {
        const float* s = stat + ((size_t)b * D + (size_t)cq * V + i) * 4;
        mh[i] = s[0]; ml[i] = s[1]; inv[i] = s[2];
    }
#pragma unroll 4
    for (int r = r0 + rl; r < r1; r += g.rl) {
        float v[V];
        ldp<V>(xb + (size_t)r * D + (size_t)cq * V, v);
#pragma unroll
        for (int i = 0; i < V; ++i) v[i] = ((v[i] - mh[i]) - ml[i]) * inv[i];
        st<V>(zb + (size_t)r * D + (size_t)cq * V, v);
    }
}

__global__ void norm_empty_kernel(int total, float* mean, float* scale) {
    kb_grid_dependency_wait();
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < total) {
        if (mean) mean[i] = 0.f;
        if (scale) scale[i] = 1.f;
    }
}

template <int V>
kb_status run(kb_ctx* ctx, int B, int N, int D, const float* x, float* z, float* mean, float* scale) {
    Geo g;
    g.cpr = D / V;
    g.cw = g.cpr < 256 ? g.cpr : 256;
    g.rl = 256 / g.cw;
    const int chunks = (g.cpr + g.cw - 1) / g.cw;
    const int G = kb_norm_blocks_per_instance(B, N);
    if (ctx->ws_bytes < kb_ws_need_normalize(B, N, D))
        return kb_fail(ctx, KB_ERR_WORKSPACE, "kb_normalize needs %zu bytes of workspace", kb_ws_need_normalize(B, N, D));
    // layout: ticket uint32[B] | stat float[B][D][4] | part double[B][G][D][2]
    size_t off_stat = kb_align256((size_t)B * 4);
    size_t off_part = off_stat + kb_align256((size_t)B * D * 4 * sizeof(float));
    float* stat = reinterpret_cast<float*>(ctx->ws + off_stat);
    double* part = reinterpret_cast<double*>(ctx->ws + off_part);
    dim3 grid(G, chunks, B);
    size_t smem = (size_t)256 * 2 * V * sizeof(double);
    kb_launch(norm_stats_kernel<V>, grid, 256, smem, ctx->stream, N, D, g, G, x, part);
    KB_LAUNCH_CHECK(ctx, "norm_stats_kernel");
    kb_launch(norm_combine_kernel, dim3((D + NC_COLS - 1) / NC_COLS, B), NC_COLS * NC_SL, 0, ctx->stream, N, D, G, x,
              static_cast<const double*>(part), stat, mean, scale);
    KB_LAUNCH_CHECK(ctx, "norm_combine_kernel");
    kb_launch(norm_apply_kernel<V>, grid, 256, 0, ctx->stream, N, D, g, G, x, z, stat);
    KB_LAUNCH_CHECK(ctx, "norm_apply_kernel");
    return KB_OK;
}

}  // namespace

size_t kb_ws_need_normalize(int B, int N, int D) {
    int G = kb_norm_blocks_per_instance(B, N);
    return kb_align256((size_t)B * 4) + kb_align256((size_t)B * D * 4 * sizeof(float)) +
           kb_align256((size_t)B * G * D * 2 * sizeof(double));
}

int kb_norm_blocks_per_instance(int B, int N) {
    // about four blocks per SM of a 148-SM part in total, at least 64 rows each
    long want = (592 + (long)B - 1) / (B > 0 ? B : 1);
    long cap = ((long)N + 63) / 64;
    if (want > cap) want = cap;
    if (want < 1) want = 1;
    if (want > KB_NORM_MAXG) want = KB_NORM_MAXG;
    return (int)want;
}

kb_status kb_launch_normalize(kb_ctx* ctx, int B, int N, int D, const float* x, float* z, float* mean,
                              float* scale) {
    if (B == 0 || D == 0) return KB_OK;
    if (N == 0) {
        if (mean || scale) {
            int total = B * D;
            kb_launch(norm_empty_kernel, (total + 255) / 256, 256, 0, ctx->stream, total, mean, scale);
            KB_LAUNCH_CHECK(ctx, "norm_empty_kernel");
        }
        return KB_OK;
    }
    if (D % 4 == 0) return run<4>(ctx, B, N, D, x, z, mean, scale);
    return run<1>(ctx, B, N, D, x, z, mean, scale);
}
