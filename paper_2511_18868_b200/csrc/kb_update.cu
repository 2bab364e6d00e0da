// kb_cluster_update: centroid = mean of its members (K-Means update, Sec. 3.3).
//
// A segmented sum by label.  Each block owns a slice of DS columns and a range
// of rows, accumulates sums[K][DS] and counts[K] in shared memory (shared
// atomics: rows of one warp instruction hit distinct banks), then flushes its
// non-zero entries to the global accumulator with one atomic each.  A second
// small kernel divides by the counts; empty clusters keep their centroid.
// X is read exactly once.  Counts are integer and exact; the fp32 sums depend
// on the order in which blocks flush (run-to-run differences in the last bits).
#include "kb_internal.cuh"

namespace {

template <int V>
__global__ void __launch_bounds__(256)
update_accum_kernel(int N, int D, int K, int DS, int G, const float* __restrict__ z,
                    const int32_t* __restrict__ labels, float* __restrict__ g_sums, int* __restrict__ g_counts,
                    int* __restrict__ dev_status) {
    extern __shared__ __align__(16) float sm[];
    float* acc = sm;                                      // [K][DS]
    int* cnt = reinterpret_cast<int*>(sm + (size_t)K * DS);  // [K]
    const int b = blockIdx.z, slice = blockIdx.y, blk = blockIdx.x;
    const int tid = threadIdx.x;
    const int sv = DS / V;                 // vectors per row in this slice
    const int rl_n = blockDim.x / sv;      // row lanes
    const int cl = tid % sv, rl = tid / sv;
    const int col = slice * DS + cl * V;   // first global column of this thread
    const bool active = rl < rl_n && col < D;
    for (int e = tid; e < K * DS + K; e += blockDim.x) sm[e] = 0.f;  // int 0 == float +0 bit pattern
    __syncthreads();

    const int rows_per = (N + G - 1) / G;
    const int r0 = blk * rows_per, r1 = min(N, r0 + rows_per);
    const float* zb = z + (size_t)b * N * D;
    const int32_t* lb = labels + (size_t)b * N;
    if (active) {
#pragma unroll 4
        for (int r = r0 + rl; r < r1; r += rl_n) {
            int lab = __ldg(lb + r);
            if (lab < 0 || lab >= K) { atomicOr(dev_status, 1); continue; }
            float* a = acc + (size_t)lab * DS + cl * V;
            if (V == 4) {
                float4 v = __ldg(reinterpret_cast<const float4*>(zb + (size_t)r * D + col));
                atomicAdd(a + 0, v.x);
                atomicAdd(a + 1, v.y);
                atomicAdd(a + 2, v.z);
                atomicAdd(a + 3, v.w);
            } else {
                atomicAdd(a, __ldg(zb + (size_t)r * D + col));
            }
            if (slice == 0 && cl == 0) atomicAdd(&cnt[lab], 1);
        }
    }
    __syncthreads();
    float* gs = g_sums + (size_t)b * K * D;
    const int width = min(DS, D - slice * DS);
    for (int e = tid; e < K * DS; e += blockDim.x) {
        int j = e / DS, c = e - j * DS;
        float v = acc[e];
        if (c < width && v != 0.f) atomicAdd(gs + (size_t)j * D + slice * DS + c, v);
    }
    if (slice == 0)
        for (int j = tid; j < K; j += blockDim.x)
            if (cnt[j]) atomicAdd(&g_counts[(size_t)b * K + j], cnt[j]);
}

__global__ void update_finalize_kernel(size_t total, int D, const float* __restrict__ g_sums,
                                       const int* __restrict__ g_counts, float* __restrict__ cent,
                                       int32_t* __restrict__ counts) {
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= total) return;
    size_t j = i / D;  // flat (b, cluster)
    int n = g_counts[j];
    if (n > 0) cent[i] = g_sums[i] / (float)n;
    if (counts && i - j * D == 0) counts[j] = n;
}

__global__ void update_empty_kernel(int total, int32_t* counts) {
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < total) counts[i] = 0;
}

int pick_ds(int D, int K, int V) {
    // largest slice (multiple of V, dividing work into equal vectors) whose K x DS tile fits ~128 KB
    long cap = (128 * 1024 / 4) / (K > 0 ? K : 1);
    long ds = D < cap ? D : cap;
    ds = ds / V * V;
    if (ds > 256 * V) ds = 256 * V;
    // a power-of-two number of vectors keeps 256 threads evenly split when possible
    if (ds >= V) {
        long sv = ds / V, p = 1;
        while (p * 2 <= sv) p *= 2;
        if ((D / V) % sv != 0 || 256 % sv != 0) ds = p * V;
    }
    return (int)ds;
}

}  // namespace

size_t kb_ws_need_update(int B, int N, int D, int K) {
    (void)N;
    return kb_align256((size_t)B * K * D * sizeof(float)) + kb_align256((size_t)B * K * sizeof(int));
}

kb_status kb_launch_update(kb_ctx* ctx, int B, int N, int D, int K, const float* z, const int32_t* labels,
                           float* c, int32_t* counts) {
    if (B == 0) return KB_OK;
    if (N == 0) {
        if (counts) {
            update_empty_kernel<<<(B * K + 255) / 256, 256, 0, ctx->stream>>>(B * K, counts);
            KB_LAUNCH_CHECK(ctx, "update_empty_kernel");
        }
        return KB_OK;
    }
    const size_t need = kb_ws_need_update(B, N, D, K);
    if (ctx->ws_bytes < need)
        return kb_fail(ctx, KB_ERR_WORKSPACE, "kb_cluster_update needs %zu bytes of workspace", need);
    float* g_sums = reinterpret_cast<float*>(ctx->ws);
    int* g_counts = reinterpret_cast<int*>(ctx->ws + kb_align256((size_t)B * K * D * sizeof(float)));
    KB_MEMSET(ctx, ctx->ws, 0, need);

    const int V = (D % 4 == 0) ? 4 : 1;
    const int DS = pick_ds(D, K, V);
    if (DS < V) return kb_fail(ctx, KB_ERR_UNSUPPORTED, "kb_cluster_update: K = %d is beyond the shared-memory path", K);
    const int slices = (D + DS - 1) / DS;
    const int threads = 256 / (DS / V) * (DS / V);
    long want = (2L * ctx->sm_count + (long)slices * B - 1) / ((long)slices * B);
    long cap = ((long)N + 255) / 256;
    int G = (int)(want < 1 ? 1 : (want > cap ? cap : want));
    size_t smem = ((size_t)K * DS + K) * sizeof(float);
    dim3 grid(G, slices, B);
    if (V == 4) {
        KB_SMEM_OPTIN(ctx, update_accum_kernel<4>, smem);
        update_accum_kernel<4><<<grid, threads, smem, ctx->stream>>>(N, D, K, DS, G, z, labels, g_sums, g_counts,
                                                                    ctx->dev_status);
    } else {
        KB_SMEM_OPTIN(ctx, update_accum_kernel<1>, smem);
        update_accum_kernel<1><<<grid, threads, smem, ctx->stream>>>(N, D, K, DS, G, z, labels, g_sums, g_counts,
                                                                    ctx->dev_status);
    }
    KB_LAUNCH_CHECK(ctx, "update_accum_kernel");
    size_t total = (size_t)B * K * D;
    update_finalize_kernel<<<(unsigned)((total + 255) / 256), 256, 0, ctx->stream>>>(total, D, g_sums, g_counts, c,
                                                                                    counts);
    KB_LAUNCH_CHECK(ctx, "update_finalize_kernel");
    return KB_OK;
}
