// kb_cluster_radius: radius[b][i] = max over the members k of cluster i of sqrt(dist2[k]).
//
// Theorem 1's regret bound carries L * max_i diam(C_i).  Through the centroid the triangle inequality
// gives diam(C_i) <= 2 radius_i, so one pass over the candidates (8 bytes each: label and distance)
// bounds the term that an exact diameter would need all pairs for.  A segmented max: non-negative
// floats order like their bit patterns, so the per-cluster maxima are integer atomicMax -- in shared
// memory per CTA, then one global atomicMax per (CTA, touched cluster) into the zeroed output.
#include "kb_internal.cuh"

namespace {

constexpr int RD_T = 256;
constexpr int RD_U = 4;
constexpr int RD_SMEM_K = 8192;   // clusters whose maxima fit the CTA's shared memory

__global__ void __launch_bounds__(RD_T)
cluster_radius_kernel(int N, int K, int rows_per, const int32_t* __restrict__ labels, const float* __restrict__ dist2,
                      float* __restrict__ radius, int* __restrict__ dev_status) {
    kb_grid_dependency_wait();
    extern __shared__ int s_max[];                     // [K] when K <= RD_SMEM_K
    const bool in_smem = K <= RD_SMEM_K;
    const int b = blockIdx.y, tid = threadIdx.x;
    if (in_smem) {
        for (int i = tid; i < K; i += RD_T) s_max[i] = 0;
        __syncthreads();
    }
    const int r0 = blockIdx.x * rows_per, r1 = min(N, r0 + rows_per);
    const int32_t* lb = labels + (size_t)b * N;
    const float* db = dist2 + (size_t)b * N;
    int* out = reinterpret_cast<int*>(radius) + (size_t)b * K;
    for (int base = r0 + tid; base < r1; base += RD_T * RD_U) {
        int lab[RD_U];
        float d[RD_U];
#pragma unroll
        for (int u = 0; u < RD_U; ++u) {
            const int r = base + u * RD_T;
            lab[u] = r < r1 ? __ldg(lb + r) : -1;
            d[u] = r < r1 ? __ldg(db + r) : 0.f;
        }
#pragma unroll
        for (int u = 0; u < RD_U; ++u) {
            if (base + u * RD_T >= r1) continue;
            if (lab[u] < 0 || lab[u] >= K) { atomicOr(dev_status, 1); continue; }
            if (!(d[u] > 0.f)) continue;               // zero, negative or NaN: nothing to add
            const int bits = __float_as_int(sqrtf(d[u]));
            if (in_smem) {
                if (bits > s_max[lab[u]]) atomicMax(&s_max[lab[u]], bits);
            } else if (bits > __ldca(out + lab[u])) {
                atomicMax(out + lab[u], bits);
            }
        }
    }
    if (in_smem) {
        __syncthreads();
        for (int i = tid; i < K; i += RD_T) {
            const int v = s_max[i];
            if (v > 0 && v > __ldca(out + i)) atomicMax(out + i, v);
        }
    }
}

}  // namespace

kb_status kb_launch_cluster_radius(kb_ctx* ctx, int B, int N, int K, const int32_t* labels, const float* dist2,
                                   float* radius) {
    if (B == 0) return KB_OK;
    KB_MEMSET(ctx, radius, 0, (size_t)B * K * sizeof(float));
    if (N == 0) return KB_OK;
    long want = (4L * ctx->sm_count + B - 1) / B;
    long cap = ((long)N + RD_T * RD_U - 1) / (RD_T * RD_U);
    long G = want < cap ? want : cap;
    if (G < 1) G = 1;
    const int rows_per = (int)((N + G - 1) / G);
    const size_t smem = K <= RD_SMEM_K ? (size_t)K * sizeof(int) : 0;
    kb_launch(cluster_radius_kernel, dim3((unsigned)G, B), RD_T, smem, ctx->stream, N, K, rows_per, labels, dist2, radius,
              ctx->dev_status);
    KB_LAUNCH_CHECK(ctx, "cluster_radius_kernel");
    return KB_OK;
}
