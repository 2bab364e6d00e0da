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
//
// When the whole K x D table of sums fits in shared memory (K*D <= 24K floats) a simpler path
// runs instead: each CTA accumulates its rows straight into a shared-memory table (shared
// atomics, rows of a warp hit different banks), writes the table out as a plain per-CTA
// partial, and the finalize kernel adds the partials in CTA order.  No global atomics, no
// memset, and the only run-to-run variation is the order of shared-memory adds inside a CTA.
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
    kb_grid_dependency_wait();
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

    // 2. Each lane group (LPR lanes = the float4 columns of one row; RPW groups per warp) takes a
    //    contiguous piece of the sorted order.  It keeps U row loads in flight regardless of where
    //    label runs end, adds the rows up in registers and flushes with one vector reduction per
    //    lane whenever the label changes.  No warp-collective operation inside a piece.
    const int LPR = (D / V) < 32 ? (D / V) : 32;                // lanes per row
    const int RPW = (32 % LPR == 0) ? 32 / LPR : 1;             // lane groups per warp
    const int lane_c = lane % LPR, lane_r = lane / LPR;
    const bool lane_on = lane_r < RPW;
    const float* zb = z + ((size_t)b * N + r0) * D;
    float* gs = g_sums + (size_t)b * K * D;
    const int npieces = (sorted + CH - 1) / CH;
    const int ngrabs = (npieces + RPW - 1) / RPW;
    constexpr int U = 8;
    for (;;) {
        int grab = 0;
        if (lane == 0) grab = atomicAdd(&s_next, 1);
        grab = __shfl_sync(0xffffffffu, grab, 0);
        if (grab >= ngrabs) break;
        const int piece = grab * RPW + lane_r;
        if (!lane_on || piece >= npieces) continue;
        const int p0 = piece * CH, p1 = min(sorted, p0 + CH);
        // label of the first position: the last j with offs[j] <= p0
        int lo = 0, hi = K - 1;
        while (lo < hi) {
            const int mid = (lo + hi + 1) >> 1;
            if (offs[mid] <= p0) lo = mid; else hi = mid - 1;
        }
        for (int cc = lane_c * V; cc < D; cc += 32 * V) {       // column chunks (one pass unless D > 32 V)
            int j = lo, jend = offs[lo + 1];
            float a[V];
#pragma unroll
            for (int i = 0; i < V; ++i) a[i] = 0.f;
            bool dirty = false;
            for (int p = p0; p < p1; p += U) {
                float v[U][V];
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    const float* src = zb + (size_t)perm[min(p + u, p1 - 1)] * D + cc;   // clamped index
                    if (V == 4) {
                        const float4 t = __ldg(reinterpret_cast<const float4*>(src));
                        v[u][0] = t.x; v[u][1 % V] = t.y; v[u][2 % V] = t.z; v[u][3 % V] = t.w;
                    } else {
                        v[u][0] = __ldg(src);
                    }
                }
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    const int pos = p + u;
                    if (pos >= p1) break;
                    if (pos >= jend) {                           // the label run ended: flush and move on
                        if (dirty) {
                            float* dst = gs + (size_t)j * D + cc;
                            if (V == 4) red_add_v4(dst, a[0], a[1 % V], a[2 % V], a[3 % V]);
                            else atomicAdd(dst, a[0]);
#pragma unroll
                            for (int i = 0; i < V; ++i) a[i] = 0.f;
                        }
                        do { ++j; jend = offs[j + 1]; } while (pos >= jend);   // skip empty labels
                    }
#pragma unroll
                    for (int i = 0; i < V; ++i) a[i] += v[u][i];
                    dirty = true;
                }
            }
            if (dirty) {
                float* dst = gs + (size_t)j * D + cc;
                if (V == 4) red_add_v4(dst, a[0], a[1 % V], a[2 % V], a[3 % V]);
                else atomicAdd(dst, a[0]);
            }
        }
    }
}

// ---- shared-memory table path ------------------------------------------------------------
constexpr int UT_T = 512;

template <int V>
__global__ void __launch_bounds__(UT_T)
update_table_kernel(int N, int D, int K, int G, const float* __restrict__ z, const int32_t* __restrict__ labels,
                    float* __restrict__ part_sums, int* __restrict__ part_cnt, int* __restrict__ dev_status) {
    kb_grid_dependency_wait();
    extern __shared__ __align__(16) float tb[];
    float* acc = tb;                                       // [K][D]
    int* cnt = reinterpret_cast<int*>(tb + (size_t)K * D); // [K]
    const int b = blockIdx.y, g = blockIdx.x, tid = threadIdx.x;
    const int KD = K * D;
    for (int e = tid; e < KD + K; e += UT_T) tb[e] = 0.f;  // int 0 == float +0 bit pattern
    __syncthreads();
    const int vpr = D / V;                                 // vectors per row
    const int rstep = UT_T / vpr;                          // rows per block step (vpr <= UT_T)
    const int rows_per = (N + G - 1) / G;
    const int r0 = g * rows_per, r1 = min(N, r0 + rows_per);
    const float* zb = z + (size_t)b * N * D;
    const int32_t* lb = labels + (size_t)b * N;
    if (tid < rstep * vpr) {
        const int q = tid % vpr;
        constexpr int U = 4;                               // rows in flight per thread
        for (int rb = r0 + tid / vpr; rb < r1; rb += U * rstep) {
            int lab[U];
            float v[U][V];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int r = min(rb + u * rstep, r1 - 1); // clamped: loads stay in range
                lab[u] = __ldg(lb + r);
                if (V == 4) {
                    const float4 t = __ldg(reinterpret_cast<const float4*>(zb + (size_t)r * D) + q);
                    v[u][0] = t.x; v[u][1 % V] = t.y; v[u][2 % V] = t.z; v[u][3 % V] = t.w;
                } else {
                    v[u][0] = __ldg(zb + (size_t)r * D + q);
                }
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                if (rb + u * rstep >= r1) break;
                if (lab[u] < 0 || lab[u] >= K) { atomicOr(dev_status, 1); continue; }
                float* a = acc + (size_t)lab[u] * D + q * V;
#pragma unroll
                for (int i = 0; i < V; ++i) atomicAdd(a + i, v[u][i]);
                if (q == 0) atomicAdd(&cnt[lab[u]], 1);
            }
        }
    }
    __syncthreads();
    float* ps = part_sums + ((size_t)b * G + g) * KD;
    for (int e = tid; e < KD; e += UT_T) ps[e] = acc[e];
    int* pc = part_cnt + ((size_t)b * G + g) * K;
    for (int j = tid; j < K; j += UT_T) pc[j] = cnt[j];
}

constexpr int UF_E = 32, UF_Y = 8;   // entries x slices of the partial index per block
__global__ void __launch_bounds__(UF_E * UF_Y)
update_table_finalize_kernel(int D, int K, int G, const float* __restrict__ part_sums,
                             const int* __restrict__ part_cnt, float* __restrict__ cent,
                             int32_t* __restrict__ counts) {
    kb_grid_dependency_wait();
    __shared__ float s_sum[UF_Y][UF_E];
    __shared__ int s_cnt[UF_Y][UF_E];
    const int b = blockIdx.y, x = threadIdx.x, y = threadIdx.y, KD = K * D;
    const int e = blockIdx.x * UF_E + x;
    // slice y adds the partials of CTAs [y*per, (y+1)*per) in order; slices are then added in order
    const int per = (G + UF_Y - 1) / UF_Y;
    float sum = 0.f;
    int n = 0;
    if (e < KD) {
        const int j = e / D;
        const int g1 = min(G, (y + 1) * per);
#pragma unroll 4
        for (int g = y * per; g < g1; ++g) {
            sum += part_sums[((size_t)b * G + g) * KD + e];
            n += part_cnt[((size_t)b * G + g) * K + j];
        }
    }
    s_sum[y][x] = sum; s_cnt[y][x] = n;
    __syncthreads();
    if (y == 0 && e < KD) {
        for (int k = 1; k < UF_Y; ++k) { sum += s_sum[k][x]; n += s_cnt[k][x]; }
        const int j = e / D;
        if (n > 0) cent[(size_t)b * KD + e] = sum / (float)n;
        if (counts && e - j * D == 0) counts[(size_t)b * K + j] = n;
    }
}

int table_ctas(int B, int N) {
    long want = (148 + (long)B - 1) / B;
    long cap = ((long)N + 255) / 256;
    long g = want < cap ? want : cap;
    return (int)(g < 1 ? 1 : g);
}
bool table_mode(int B, int N, int D, int K) {
    // shared-memory float atomics are slow; worth it only where launch count dominates
    return (long)B * N <= 32768 && (long)K * D <= 24 * 1024 && (D % 4 == 0 ? D / 4 : D) <= UT_T;
}

__global__ void update_finalize_kernel(size_t total, int D, const float* __restrict__ g_sums,
                                       const int* __restrict__ g_counts, float* __restrict__ cent,
                                       int32_t* __restrict__ counts) {
    kb_grid_dependency_wait();
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= total) return;
    size_t j = i / D;  // flat (b, cluster)
    int n = g_counts[j];
    if (n > 0) cent[i] = g_sums[i] / (float)n;
    if (counts && i - j * D == 0) counts[j] = n;
}

// clears the accumulators (a kernel rather than a memset node, so that it chains with its
// neighbours by programmatic dependent launch)
__global__ void update_zero_kernel(size_t n16, uint4* __restrict__ p) {
    kb_grid_dependency_wait();
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n16) p[i] = make_uint4(0u, 0u, 0u, 0u);
}

__global__ void update_empty_kernel(int total, int32_t* counts) {
    kb_grid_dependency_wait();
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < total) counts[i] = 0;
}

}  // namespace

size_t kb_ws_need_update(int B, int N, int D, int K) {
    size_t need = kb_align256((size_t)B * K * D * sizeof(float)) + kb_align256((size_t)B * K * sizeof(int));
    if (table_mode(B, N, D, K)) {
        const size_t G = table_ctas(B, N);
        const size_t t = kb_align256((size_t)B * G * K * D * sizeof(float)) + kb_align256((size_t)B * G * K * sizeof(int));
        if (t > need) need = t;
    }
    return need;
}

// A fit's own accumulators: sums [B][K][D], then counts [B][K].
size_t kb_ws_need_fit_acc(int B, int D, int K) {
    return kb_align256((size_t)B * K * D * sizeof(float)) + kb_align256((size_t)B * K * sizeof(int));
}

kb_status kb_launch_update(kb_ctx* ctx, int B, int N, int D, int K, const float* z, const int32_t* labels,
                           float* c, int32_t* counts) {
    if (B == 0) return KB_OK;
    if (N == 0) {
        if (counts) {
            kb_launch(update_empty_kernel, (B * K + 255) / 256, 256, 0, ctx->stream, B * K, counts);
            KB_LAUNCH_CHECK(ctx, "update_empty_kernel");
        }
        return KB_OK;
    }
    const size_t need = kb_ws_need_update(B, N, D, K);
    if (ctx->ws_bytes < need)
        return kb_fail(ctx, KB_ERR_WORKSPACE, "kb_cluster_update needs %zu bytes of workspace", need);
    if (table_mode(B, N, D, K)) {
        const int G = table_ctas(B, N);
        float* part_sums = reinterpret_cast<float*>(ctx->ws);
        int* part_cnt = reinterpret_cast<int*>(ctx->ws + kb_align256((size_t)B * G * K * D * sizeof(float)));
        const size_t smem = ((size_t)K * D + K) * sizeof(float);
        if (D % 4 == 0) {
            KB_SMEM_OPTIN(ctx, update_table_kernel<4>, smem);
            kb_launch(update_table_kernel<4>, dim3(G, B), UT_T, smem, ctx->stream, N, D, K, G, z, labels, part_sums, part_cnt,
                                                                         ctx->dev_status);
        } else {
            KB_SMEM_OPTIN(ctx, update_table_kernel<1>, smem);
            kb_launch(update_table_kernel<1>, dim3(G, B), UT_T, smem, ctx->stream, N, D, K, G, z, labels, part_sums, part_cnt,
                                                                         ctx->dev_status);
        }
        KB_LAUNCH_CHECK(ctx, "update_table_kernel");
        kb_launch(update_table_finalize_kernel, dim3((K * D + UF_E - 1) / UF_E, B), dim3(UF_E, UF_Y), 0, ctx->stream, 
            D, K, G, part_sums, part_cnt, c, counts);
        KB_LAUNCH_CHECK(ctx, "update_table_finalize_kernel");
        return KB_OK;
    }
    // inside a tensor-path fit the accumulators are the fit's own, already cleared by the assignment before
    const bool own = ctx->fit_acc && ctx->fit_acc_clean && ctx->fit_acc_bytes == kb_ws_need_fit_acc(B, D, K);
    char* acc = own ? ctx->fit_acc : ctx->ws;
    float* g_sums = reinterpret_cast<float*>(acc);
    int* g_counts = reinterpret_cast<int*>(acc + kb_align256((size_t)B * K * D * sizeof(float)));
    if (own) {
        ctx->fit_acc_clean = 0;
    } else {
        kb_launch(update_zero_kernel, (unsigned)((need / 16 + 255) / 256), 256, 0, ctx->stream, need / 16,
                  reinterpret_cast<uint4*>(ctx->ws));
        KB_LAUNCH_CHECK(ctx, "update_zero_kernel");
    }

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
    // piece of the sorted order a lane group takes at a time: about four pieces per group, 8..128 positions
    const int groups = (UP_T / 32) * rpw;
    int CH = (rows_per + 4 * groups - 1) / (4 * groups);
    CH = CH < 8 ? 8 : (CH > 128 ? 128 : CH);
    dim3 grid((unsigned)G, B);
    if (V == 4) {
        KB_SMEM_OPTIN(ctx, update_sorted_kernel<4>, smem);
        kb_launch(update_sorted_kernel<4>, grid, UP_T, smem, ctx->stream, N, D, K, (int)G, CH, z, labels, g_sums, g_counts,
                                                                  ctx->dev_status);
    } else {
        KB_SMEM_OPTIN(ctx, update_sorted_kernel<1>, smem);
        kb_launch(update_sorted_kernel<1>, grid, UP_T, smem, ctx->stream, N, D, K, (int)G, CH, z, labels, g_sums, g_counts,
                                                                  ctx->dev_status);
    }
    KB_LAUNCH_CHECK(ctx, "update_sorted_kernel");
    size_t total = (size_t)B * K * D;
    kb_launch(update_finalize_kernel, (unsigned)((total + 255) / 256), 256, 0, ctx->stream, total, D, g_sums, g_counts, c,
                                                                                    counts);
    KB_LAUNCH_CHECK(ctx, "update_finalize_kernel");
    return KB_OK;
}

// ---- centroid update for callers that must not allocate ------------------------------------
// Scratch for kb_cluster_update_noalloc lives in the library image itself: one file-scope
// device array, present on every GPU that loads the library until the process exits.
// Layout: [0, 256) status word | sums float[KB_NOALLOC_MAX_KD] | counts int[KB_NOALLOC_MAX_K].
#define KB_NOALLOC_SCRATCH_BYTES (256 + (size_t)KB_NOALLOC_MAX_KD * sizeof(float) + (size_t)KB_NOALLOC_MAX_K * sizeof(int))
static __device__ __align__(256) unsigned char kb_noalloc_scratch[KB_NOALLOC_SCRATCH_BYTES];

namespace {
constexpr int NOALLOC_MAX_DEVICES = 64;
// Device address of the array above, per device.  In host code the array's NAME is only a
// stand-in for the symbol, not a device pointer, so the address is asked for once per
// device with cudaGetSymbolAddress and remembered here.
void* g_noalloc_ptr[NOALLOC_MAX_DEVICES];
int g_noalloc_sms[NOALLOC_MAX_DEVICES];
int g_noalloc_smem[NOALLOC_MAX_DEVICES];
}  // namespace

// Set-up of the current device, once: the scratch array's device address and two attributes.
// Two threads that race here write the same values (the look-up is idempotent).
static kb_status noalloc_setup(int* dev_out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= NOALLOC_MAX_DEVICES) return KB_ERR_CUDA;
    if (!g_noalloc_ptr[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, kb_noalloc_scratch) != cudaSuccess || !p) return KB_ERR_CUDA;
        if (cudaDeviceGetAttribute(&g_noalloc_sms[dev], cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&g_noalloc_smem[dev], cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess)
            return KB_ERR_CUDA;
        g_noalloc_ptr[dev] = p;
    }
    *dev_out = dev;
    return KB_OK;
}

extern "C" kb_status kb_cluster_update_noalloc_status(void* cuda_stream, int* out) {
    if (!out) return KB_ERR_INVALID_ARG;
    int dev = -1;
    const kb_status s = noalloc_setup(&dev);
    if (s != KB_OK) return s;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    int word = 0;
    if (cudaMemcpyAsync(&word, g_noalloc_ptr[dev], sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess) return KB_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return KB_ERR_CUDA;
    if (word != 0 && cudaMemsetAsync(g_noalloc_ptr[dev], 0, sizeof(int), st) != cudaSuccess) return KB_ERR_CUDA;
    *out = word;
    return KB_OK;
}

extern "C" kb_status kb_cluster_update_noalloc(void* cuda_stream, int N, int D, int K, const float* z,
                                               const int32_t* labels, float* centroids, int32_t* counts) {
    if (N < 0 || D < 1 || K < 1) return KB_ERR_INVALID_ARG;
    if (!centroids || (N > 0 && (!z || !labels))) return KB_ERR_INVALID_ARG;
    if (D % 4 == 0 && (((uintptr_t)z) & 15) != 0) return KB_ERR_INVALID_ARG;
    // sizes beyond the built-in scratch are refused, never truncated
    if ((long long)K * D > KB_NOALLOC_MAX_KD || K > KB_NOALLOC_MAX_K) return KB_ERR_UNSUPPORTED;
    int dev = -1;
    const kb_status su = noalloc_setup(&dev);      // first call on this device (it is the current one)
    if (su != KB_OK) return su;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    unsigned char* base = static_cast<unsigned char*>(g_noalloc_ptr[dev]);
    int* status = reinterpret_cast<int*>(base);
    float* g_sums = reinterpret_cast<float*>(base + 256);
    int* g_counts = reinterpret_cast<int*>(base + 256 + (size_t)KB_NOALLOC_MAX_KD * sizeof(float));
    if (N == 0) {
        if (counts) {
            update_empty_kernel<<<(K + 255) / 256, 256, 0, st>>>(K, counts);
            if (cudaGetLastError() != cudaSuccess) return KB_ERR_CUDA;
        }
        return KB_OK;
    }
    // the array keeps whatever the previous call left: clear the part this call accumulates into
    if (cudaMemsetAsync(g_sums, 0, (size_t)K * D * sizeof(float), st) != cudaSuccess) return KB_ERR_CUDA;
    if (cudaMemsetAsync(g_counts, 0, (size_t)K * sizeof(int), st) != cudaSuccess) return KB_ERR_CUDA;
    long want = 2L * g_noalloc_sms[dev];
    long lo = ((long)N + UP_MAXROWS - 1) / UP_MAXROWS;
    long hi = ((long)N + 511) / 512;
    long G = want < lo ? lo : want;
    if (G > hi) G = hi;
    if (G < lo) G = lo;
    if (G < 1) G = 1;
    const int rows_per = (int)((N + G - 1) / G);
    const size_t smem = ((size_t)2 * K + 1) * sizeof(int) + (size_t)rows_per * sizeof(unsigned short) + 16;
    if (smem > (size_t)g_noalloc_smem[dev] - 256) return KB_ERR_UNSUPPORTED;
    const int V = (D % 4 == 0) ? 4 : 1;
    const int lpr = (D / V) < 32 ? (D / V) : 32;
    const int rpw = (32 % lpr == 0) ? 32 / lpr : 1;
    const int groups = (UP_T / 32) * rpw;
    int CH = (rows_per + 4 * groups - 1) / (4 * groups);
    CH = CH < 8 ? 8 : (CH > 128 ? 128 : CH);
    dim3 grid((unsigned)G, 1);
    if (V == 4) {
        if (smem > 48 * 1024 &&
            cudaFuncSetAttribute(update_sorted_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
            return KB_ERR_CUDA;
        update_sorted_kernel<4><<<grid, UP_T, smem, st>>>(N, D, K, (int)G, CH, z, labels, g_sums, g_counts, status);
    } else {
        if (smem > 48 * 1024 &&
            cudaFuncSetAttribute(update_sorted_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
            return KB_ERR_CUDA;
        update_sorted_kernel<1><<<grid, UP_T, smem, st>>>(N, D, K, (int)G, CH, z, labels, g_sums, g_counts, status);
    }
    if (cudaGetLastError() != cudaSuccess) return KB_ERR_CUDA;
    const size_t total = (size_t)K * D;
    update_finalize_kernel<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(total, D, g_sums, g_counts, centroids, counts);
    if (cudaGetLastError() != cudaSuccess) return KB_ERR_CUDA;
    return KB_OK;
}
