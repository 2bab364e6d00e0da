// kb_cluster_update: centroid = mean of its members (K-Means update, Sec. 3.3).
//
// A segmented sum by label that reads X exactly once and keeps float atomics out
// of the inner loop.  Each CTA owns a contiguous range of rows of one instance:
//   1. counting sort of its rows by label in shared memory (integer shared
//      atomics only: histogram, exclusive scan, scatter of 16-bit local row ids);
//   2. warps grab chunks of the sorted order and add up the rows of one label at a
//      time in registers (lane = float4 column, several rows in flight per warp);
//   3. one vector reduction (red.global.add.v4.f32) per (chunk, label) run into the
//      global accumulator; integer counts are flushed once per CTA and are exact.
// A second small kernel divides by the counts; empty clusters keep their centroid.
// The fp32 sums depend on the order in which runs are flushed (last-bit
// run-to-run differences); counts never do.
#include "kb_internal.cuh"

namespace {

constexpr int UP_T = 512;          // threads per CTA
constexpr int UP_MAXROWS = 32768;  // rows per CTA (16-bit local ids)

__device__ __forceinline__ void red_add_v4(float* addr, float a, float b, float c, float d) {
    asm volatile("red.relaxed.gpu.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(addr), "f"(a), "f"(b), "f"(c), "f"(d)
                 : "memory");
}

template <int V>
__global__ void __launch_bounds__(UP_T)
update_sorted_kernel(int N, int D, int K, int G, int CH, const float* __restrict__ z,
                     const int32_t* __restrict__ labels, float* __restrict__ g_sums, int* __restrict__ g_counts,
                     int* __restrict__ dev_status) {
    extern __shared__ __align__(16) unsigned char sm_raw[];
    int* hist = reinterpret_cast<int*>(sm_raw);                // [K]  counts, then scatter cursors
    int* offs = hist + K;                                      // [K+1] exclusive prefix
    unsigned short* perm = reinterpret_cast<unsigned short*>(offs + K + 1);   // [rows] local row ids in label order
    __shared__ int s_warp_tot[UP_T / 32];
    __shared__ int s_next;
    const int b = blockIdx.y, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int rows_per = (N + G - 1) / G;
    const int r0 = blockIdx.x * rows_per;
    const int rows = max(0, min(N, r0 + rows_per) - r0);
    const int32_t* lb = labels + (size_t)b * N + r0;

    for (int j = tid; j < K; j += UP_T) hist[j] = 0;
    if (tid == 0) s_next = 0;
    __syncthreads();
    // 1a. histogram
    for (int r = tid; r < rows; r += UP_T) {
        const int lab = __ldg(lb + r);
        if (lab < 0 || lab >= K) { atomicOr(dev_status, 1); continue; }
        atomicAdd(&hist[lab], 1);
    }
    __syncthreads();
    // 1b. exclusive scan of hist -> offs (each thread scans a contiguous slice), counts to global
    {
        const int per = (K + UP_T - 1) / UP_T;
        const int j0 = min(K, tid * per), j1 = min(K, j0 + per);
        int local = 0;
        for (int j = j0; j < j1; ++j) local += hist[j];
        int incl = local;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            int v = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += v;
        }
        if (lane == 31) s_warp_tot[warp] = incl;
        __syncthreads();
        int base = 0;
        for (int w = 0; w < warp; ++w) base += s_warp_tot[w];
        int run = base + incl - local;
        for (int j = j0; j < j1; ++j) {
            const int c = hist[j];
            offs[j] = run;
            if (c) atomicAdd(&g_counts[(size_t)b * K + j], c);
            run += c;
        }
        if (tid == UP_T - 1) offs[K] = run;
    }
    __syncthreads();
    for (int j = tid; j < K; j += UP_T) hist[j] = offs[j];      // scatter cursors
    __syncthreads();
    // 1c. scatter local row ids into label order
    for (int r = tid; r < rows; r += UP_T) {
        const int lab = __ldg(lb + r);
        if (lab < 0 || lab >= K) continue;
        const int pos = atomicAdd(&hist[lab], 1);
        perm[pos] = (unsigned short)r;
    }
    __syncthreads();
    const int sorted = offs[K];                                 // rows with a valid label

    // 2. chunks of the sorted order, one label run at a time
    const int LPR = (D / V) < 32 ? (D / V) : 32;                // lanes per row
    const int RPW = (32 % LPR == 0) ? 32 / LPR : 1;             // rows in flight per warp step
    const int lane_c = lane % LPR, lane_r = lane / LPR;
    const bool lane_on = lane_r < RPW;
    const float* zb = z + ((size_t)b * N + r0) * D;
    float* gs = g_sums + (size_t)b * K * D;
    const int nchunks = (sorted + CH - 1) / CH;
    for (;;) {
        int chunk = 0;
        if (lane == 0) chunk = atomicAdd(&s_next, 1);
        chunk = __shfl_sync(0xffffffffu, chunk, 0);
        if (chunk >= nchunks) break;
        const int p0 = chunk * CH, p1 = min(sorted, p0 + CH);
        // first label of the chunk: the last j with offs[j] <= p0
        int lo = 0, hi = K - 1;
        while (lo < hi) {
            const int mid = (lo + hi + 1) >> 1;
            if (offs[mid] <= p0) lo = mid; else hi = mid - 1;
        }
        int j = lo, p = p0;
        while (p < p1) {
            while (offs[j + 1] <= p) ++j;                        // skip empty labels
            const int pe = min(p1, offs[j + 1]);
            for (int cc = lane_c * V; cc < D; cc += 32 * V) {    // column chunks (one pass unless D > 32 V)
                float a[V];
#pragma unroll
                for (int i = 0; i < V; ++i) a[i] = 0.f;
                if (lane_on) {
                    int q = p + lane_r;
#pragma unroll 1
                    for (; q + 3 * RPW < pe; q += 4 * RPW) {     // four independent rows in flight per lane
                        const float* s0 = zb + (size_t)perm[q] * D + cc;
                        const float* s1 = zb + (size_t)perm[q + RPW] * D + cc;
                        const float* s2 = zb + (size_t)perm[q + 2 * RPW] * D + cc;
                        const float* s3 = zb + (size_t)perm[q + 3 * RPW] * D + cc;
                        if (V == 4) {
                            const float4 v0 = __ldg(reinterpret_cast<const float4*>(s0));
                            const float4 v1 = __ldg(reinterpret_cast<const float4*>(s1));
                            const float4 v2 = __ldg(reinterpret_cast<const float4*>(s2));
                            const float4 v3 = __ldg(reinterpret_cast<const float4*>(s3));
                            a[0] += (v0.x + v1.x) + (v2.x + v3.x);
                            a[1 % V] += (v0.y + v1.y) + (v2.y + v3.y);
                            a[2 % V] += (v0.z + v1.z) + (v2.z + v3.z);
                            a[3 % V] += (v0.w + v1.w) + (v2.w + v3.w);
                        } else {
                            a[0] += (__ldg(s0) + __ldg(s1)) + (__ldg(s2) + __ldg(s3));
                        }
                    }
                    for (; q < pe; q += RPW) {
                        const float* s0 = zb + (size_t)perm[q] * D + cc;
                        if (V == 4) {
                            const float4 v0 = __ldg(reinterpret_cast<const float4*>(s0));
                            a[0] += v0.x; a[1 % V] += v0.y; a[2 % V] += v0.z; a[3 % V] += v0.w;
                        } else {
                            a[0] += __ldg(s0);
                        }
                    }
                }
                // fold the rows that ran in parallel lanes
                for (int o = LPR; o < LPR * RPW; o <<= 1) {
#pragma unroll
                    for (int i = 0; i < V; ++i) a[i] += __shfl_xor_sync(0xffffffffu, a[i], o);
                }
                if (lane < LPR && cc < D) {
                    float* dst = gs + (size_t)j * D + cc;
                    if (V == 4) red_add_v4(dst, a[0], a[1 % V], a[2 % V], a[3 % V]);
                    else atomicAdd(dst, a[0]);
                }
            }
            p = pe;
        }
    }
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

    // CTAs per instance: about two per SM in total, each with at most UP_MAXROWS rows and
    // enough rows to be worth a sort
    long want = (2L * ctx->sm_count + B - 1) / B;
    long lo = ((long)N + UP_MAXROWS - 1) / UP_MAXROWS;
    long hi = ((long)N + 511) / 512;
    long G = want < lo ? lo : want;
    if (G > hi) G = hi;
    if (G < lo) G = lo;
    if (G < 1) G = 1;
    const int rows_per = (int)((N + G - 1) / G);
    const size_t smem = ((size_t)2 * K + 1) * sizeof(int) + (size_t)rows_per * sizeof(unsigned short) + 16;
    if (smem > (size_t)ctx->max_smem_optin - 256)
        return kb_fail(ctx, KB_ERR_UNSUPPORTED, "kb_cluster_update: K = %d is beyond the shared-memory path", K);
    const int V = (D % 4 == 0) ? 4 : 1;
    const int lpr = (D / V) < 32 ? (D / V) : 32;
    const int rpw = (32 % lpr == 0) ? 32 / lpr : 1;
    // chunk of the sorted order a warp takes at a time: about four chunks per warp, 32..256 positions
    int CH = (rows_per + 4 * (UP_T / 32) - 1) / (4 * (UP_T / 32));
    CH = CH < 32 ? 32 : (CH > 256 ? 256 : CH);
    CH = (CH + rpw - 1) / rpw * rpw;
    dim3 grid((unsigned)G, B);
    if (V == 4) {
        KB_SMEM_OPTIN(ctx, update_sorted_kernel<4>, smem);
        update_sorted_kernel<4><<<grid, UP_T, smem, ctx->stream>>>(N, D, K, (int)G, CH, z, labels, g_sums, g_counts,
                                                                  ctx->dev_status);
    } else {
        KB_SMEM_OPTIN(ctx, update_sorted_kernel<1>, smem);
        update_sorted_kernel<1><<<grid, UP_T, smem, ctx->stream>>>(N, D, K, (int)G, CH, z, labels, g_sums, g_counts,
                                                                  ctx->dev_status);
    }
    KB_LAUNCH_CHECK(ctx, "update_sorted_kernel");
    size_t total = (size_t)B * K * D;
    update_finalize_kernel<<<(unsigned)((total + 255) / 256), 256, 0, ctx->stream>>>(total, D, g_sums, g_counts, c,
                                                                                    counts);
    KB_LAUNCH_CHECK(ctx, "update_finalize_kernel");
    return KB_OK;
}
