// kb_seed_kmeanspp: k-means++ seeding (Arthur & Vassilvitskii, SODA'07), the initialisation behind the
// "scikit-learn's KMeans" of Sec. 3.5 (without its extra greedy trials).
//
// The first centre is a row drawn uniformly; every further centre is a row drawn with probability
// D(x)^2 / sum D^2, D(x) = distance to the nearest centre chosen so far.  Each draw is a Gumbel-max
// over the weights (row with the largest ln(w) + G, G = -ln(-ln u)): one pass over the rows per
// round, no prefix sum over the weights and no second pass to locate the drawn row.  u comes from
// Philox4x32-10 at counter (row, instance, round, 1), so the draw does not depend on the launch shape.
//
// One launch per round.  A round reads Z once (plus the row chosen in the previous round), keeps
// min D^2 per row in scratch (4 bytes per row read and written), and reduces two packed keys per
// instance: the weighted draw, and a uniform draw that is used only when every weight is zero
// (fewer distinct rows than K).  The last CTA of an instance to finish writes the round's row.
#include "kb_internal.cuh"

namespace {

constexpr int SD_T = 256;

struct SeedWs {
    unsigned long long* key;   // [B][K][2]  weighted draw, uniform draw
    unsigned* done;            // [B][K]
    float* mind2;              // [B][N]
};

size_t seed_carve(char* ws, int B, int N, int K, SeedWs* out, size_t* zero_bytes) {
    size_t o = 0;
    SeedWs w;
    w.key = reinterpret_cast<unsigned long long*>(ws + o);  o += kb_align256((size_t)B * K * 16);
    w.done = reinterpret_cast<unsigned*>(ws + o);           o += kb_align256((size_t)B * K * 4);
    if (zero_bytes) *zero_bytes = o;
    w.mind2 = reinterpret_cast<float*>(ws + o);             o += kb_align256((size_t)B * N * 4);
    if (out) *out = w;
    return o;
}

__device__ __forceinline__ unsigned long long seed_pack(float v, int r) {
    return ((unsigned long long)kb_orderable(v) << 32) | (unsigned long long)(0xffffffffu - (unsigned)r);
}

template <int V>
__global__ void __launch_bounds__(SD_T)
seed_round_kernel(int N, int D, int K, int round, int G, int rows_per, const float* __restrict__ z,
                  int32_t* __restrict__ rows, uint32_t seed_lo, uint32_t seed_hi, SeedWs w) {
    kb_grid_dependency_wait();
    __shared__ unsigned long long s_red[2][SD_T / 32];
    const int b = blockIdx.y, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int vpr = D / V;                                       // vectors per row
    const int lpr = vpr >= 32 ? 32 : (32 % vpr == 0 ? vpr : 32); // lanes per row
    const int rpw = 32 / lpr;                                    // rows per warp step
    const int lane_c = lane % lpr, lane_r = lane / lpr;
    const int r0 = blockIdx.x * rows_per, r1 = min(N, r0 + rows_per);
    const float* zb = z + (size_t)b * N * D;
    float* md = w.mind2 + (size_t)b * N;
    const int c = round > 0 ? rows[(size_t)b * K + round - 1] : 0;
    const float* zc = zb + (size_t)c * D;
    unsigned long long bestW = 0ull, bestU = 0ull;
    constexpr int U = 4;
    __shared__ float s_d2[SD_T / 32][32];
    // A warp takes 32 consecutive rows per trip.  Phase 1: lane groups (lpr lanes = the columns of a row) form the
    // squared distance to the newest centre, U row loads in flight per lane, and leave it in shared memory.
    // Phase 2: one row per lane -- min with the stored weight (coalesced), the generator, the logarithms, the keys.
    // The trip count is the same for every thread of the block; rows past the end are computed on the last row
    // and dropped in phase 2.
    const int trips = (max(r1 - r0, 0) + SD_T - 1) / SD_T;
    for (int it = 0; it < trips; ++it) {
        const int base = r0 + (it * (SD_T / 32) + warp) * 32;
        if (round > 0) {
            for (int v0 = 0; v0 < 32 / rpw; v0 += U) {
                float acc[U];
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    const int r = min(base + (v0 + u) * rpw + lane_r, r1 - 1);
                    const float* x = zb + (size_t)r * D;
                    float a = 0.f;
                    for (int q = lane_c; q < vpr; q += lpr) {
                        if (V == 4) {
                            const float4 xv = __ldg(reinterpret_cast<const float4*>(x) + q);
                            const float4 cv = __ldg(reinterpret_cast<const float4*>(zc) + q);
                            const float e0 = xv.x - cv.x, e1 = xv.y - cv.y, e2 = xv.z - cv.z, e3 = xv.w - cv.w;
                            a = fmaf(e0, e0, a); a = fmaf(e1, e1, a); a = fmaf(e2, e2, a); a = fmaf(e3, e3, a);
                        } else {
                            const float e = __ldg(x + q) - __ldg(zc + q);
                            a = fmaf(e, e, a);
                        }
                    }
                    acc[u] = a;
                }
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    float a = acc[u];
                    for (int o = 1; o < lpr; o <<= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
                    if (lane_c == 0 && v0 + u < 32 / rpw) s_d2[warp][(v0 + u) * rpw + lane_r] = a;   // (narrow rows: fewer than U steps)
                }
            }
            __syncwarp();
        }
        const int r = base + lane;
        if (r < r1) {
            float wgt = 1.f;
            if (round > 0) {
                const float a = s_d2[warp][lane];
                wgt = round == 1 ? a : fminf(md[r], a);
                if (round + 1 < K) md[r] = wgt;
            }
            const uint32_t w0 = kb_philox4x32_10_word0((uint32_t)r, (uint32_t)b, (uint32_t)round, 1u, seed_lo, seed_hi);
            const float g = -logf(-logf(kb_uniform23(w0)));
            const unsigned long long ku = seed_pack(g, r);
            bestU = ku > bestU ? ku : bestU;
            if (wgt > 0.f) {
                const unsigned long long kw = seed_pack(logf(wgt) + g, r);
                bestW = kw > bestW ? kw : bestW;
            }
        }
        __syncwarp();                                           // s_d2 is rewritten by the next trip
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const unsigned long long a = __shfl_xor_sync(0xffffffffu, bestW, o);
        const unsigned long long u = __shfl_xor_sync(0xffffffffu, bestU, o);
        bestW = a > bestW ? a : bestW;
        bestU = u > bestU ? u : bestU;
    }
    if (lane == 0) { s_red[0][warp] = bestW; s_red[1][warp] = bestU; }
    __syncthreads();
    if (tid != 0) return;
#pragma unroll
    for (int i = 1; i < SD_T / 32; ++i) {
        bestW = s_red[0][i] > bestW ? s_red[0][i] : bestW;
        bestU = s_red[1][i] > bestU ? s_red[1][i] : bestU;
    }
    const size_t slot = (size_t)b * K + round;
    if (G > 1) {
        if (bestW) atomicMax(&w.key[2 * slot], bestW);
        if (bestU) atomicMax(&w.key[2 * slot + 1], bestU);
        __threadfence();
        if (atomicAdd(&w.done[slot], 1u) != (unsigned)G - 1u) return;
        __threadfence();
        bestW = atomicMax(&w.key[2 * slot], 0ull);
        bestU = atomicMax(&w.key[2 * slot + 1], 0ull);
    }
    const unsigned long long k = bestW ? bestW : bestU;          // every weight zero: the uniform draw
    rows[slot] = (int32_t)(0xffffffffu - (unsigned)(k & 0xffffffffull));
}

// Small instances (at most SD_T * SD_R rows): all K rounds in one launch, one CTA per instance.  A thread owns up
// to SD_R rows and keeps their weights in registers; the rows are re-read every round (the instance stays in L1/L2),
// each round ends in two block maxima (weighted and uniform draw) instead of atomics and a ticket.
// STAGE: the instance is first copied into shared memory (rows padded by four floats, so that a warp's float4 reads
// of 32 different rows meet no bank twice) and every round reads it from there; without it the K re-reads of all
// instances in flight go to L2, which then bounds the kernel.
constexpr int SD_R = 4;

__device__ __forceinline__ unsigned long long seed_block_max(unsigned long long v, unsigned long long* s_red) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const unsigned long long other = __shfl_xor_sync(0xffffffffu, v, o);
        v = other > v ? other : v;
    }
    __syncthreads();                                             // s_red may still be read from the reduction before
    if ((threadIdx.x & 31) == 0) s_red[threadIdx.x >> 5] = v;
    __syncthreads();
    v = s_red[0];
#pragma unroll
    for (int w = 1; w < SD_T / 32; ++w) v = s_red[w] > v ? s_red[w] : v;
    return v;
}

template <int V, bool STAGE>
__global__ void __launch_bounds__(SD_T)
seed_small_kernel(int N, int D, int K, const float* __restrict__ z, int32_t* __restrict__ rows, uint32_t seed_lo,
                  uint32_t seed_hi) {
    kb_grid_dependency_wait();
    extern __shared__ __align__(16) float s_z[];                 // STAGE: [N][D + 4]
    __shared__ unsigned long long s_red[SD_T / 32];
    const int b = blockIdx.x, tid = threadIdx.x;
    const float* zg = z + (size_t)b * N * D;
    const int ld = STAGE ? D + 4 : D;                            // floats between two rows
    if (STAGE) {
        const int vpr = D / 4;
        for (int e = tid; e < N * vpr; e += SD_T) {
            const int r = e / vpr, q = e - r * vpr;
            *reinterpret_cast<float4*>(s_z + (size_t)r * ld + 4 * q) = __ldg(reinterpret_cast<const float4*>(zg) + e);
        }
        __syncthreads();
    }
    const float* zb = STAGE ? s_z : zg;
    float wgt[SD_R];
#pragma unroll
    for (int j = 0; j < SD_R; ++j) wgt[j] = 1.f;
    int c = 0;
    for (int round = 0; round < K; ++round) {
        unsigned long long bestW = 0ull, bestU = 0ull;
        const float* zc = zb + (size_t)c * ld;
#pragma unroll
        for (int j = 0; j < SD_R; ++j) {
            const int r = tid + j * SD_T;
            if (r >= N) continue;
            if (round > 0) {
                const float* x = zb + (size_t)r * ld;
                float a = 0.f;
                if (V == 4) {
                    for (int q = 0; q < D / 4; ++q) {
                        const float4 xv = STAGE ? reinterpret_cast<const float4*>(x)[q] : __ldg(reinterpret_cast<const float4*>(x) + q);
                        const float4 cv = STAGE ? reinterpret_cast<const float4*>(zc)[q] : __ldg(reinterpret_cast<const float4*>(zc) + q);
                        const float e0 = xv.x - cv.x, e1 = xv.y - cv.y, e2 = xv.z - cv.z, e3 = xv.w - cv.w;
                        a = fmaf(e0, e0, a); a = fmaf(e1, e1, a); a = fmaf(e2, e2, a); a = fmaf(e3, e3, a);
                    }
                } else {
                    for (int q = 0; q < D; ++q) {
                        const float e = __ldg(x + q) - __ldg(zc + q);
                        a = fmaf(e, e, a);
                    }
                }
                wgt[j] = round == 1 ? a : fminf(wgt[j], a);
            }
            const uint32_t w0 = kb_philox4x32_10_word0((uint32_t)r, (uint32_t)b, (uint32_t)round, 1u, seed_lo, seed_hi);
            const float g = -logf(-logf(kb_uniform23(w0)));
            const unsigned long long ku = seed_pack(g, r);
            bestU = ku > bestU ? ku : bestU;
            if (wgt[j] > 0.f) {
                const unsigned long long kw = seed_pack(logf(wgt[j]) + g, r);
                bestW = kw > bestW ? kw : bestW;
            }
        }
        bestW = seed_block_max(bestW, s_red);
        if (bestW == 0ull) bestW = seed_block_max(bestU, s_red);   // every weight zero (uniform over the block): the uniform draw
        c = (int)(0xffffffffu - (unsigned)(bestW & 0xffffffffull));
        if (tid == 0) rows[(size_t)b * K + round] = c;
    }
}

int seed_ctas(const kb_ctx* ctx, int B, int N) {
    long want = (4L * ctx->sm_count + B - 1) / B;
    long cap = ((long)N + SD_T - 1) / SD_T;                      // at least one trip of rows per CTA
    long g = want < cap ? want : cap;
    return (int)(g < 1 ? 1 : g);
}

}  // namespace

size_t kb_ws_need_seed(int B, int N, int K) {
    if (B < 1 || N < 1 || K < 1) return 0;
    return seed_carve(nullptr, B, N, K, nullptr, nullptr);
}

kb_status kb_launch_seed_kmeanspp(kb_ctx* ctx, int B, int N, int D, int K, const float* z, uint64_t seed,
                                  int32_t* rows) {
    if (B == 0) return KB_OK;
    const bool vec = (D % 4 == 0) && (((uintptr_t)z & 15) == 0);
    const uint32_t s_lo = (uint32_t)(seed & 0xffffffffu), s_hi = (uint32_t)(seed >> 32);
    if (N <= SD_T * SD_R && (long)B * 2 >= ctx->sm_count) {
        // many small instances: every round of an instance in one CTA, one launch in all
        const size_t stage = (size_t)N * (D + 4) * sizeof(float);
        if (vec && stage + 1024 <= (size_t)ctx->max_smem_optin) {
            KB_SMEM_OPTIN(ctx, (seed_small_kernel<4, true>), stage);
            kb_launch((seed_small_kernel<4, true>), B, SD_T, stage, ctx->stream, N, D, K, z, rows, s_lo, s_hi);
        } else if (vec) {
            kb_launch((seed_small_kernel<4, false>), B, SD_T, 0, ctx->stream, N, D, K, z, rows, s_lo, s_hi);
        } else {
            kb_launch((seed_small_kernel<1, false>), B, SD_T, 0, ctx->stream, N, D, K, z, rows, s_lo, s_hi);
        }
        KB_LAUNCH_CHECK(ctx, "seed_small_kernel");
        return KB_OK;
    }
    const size_t need = kb_ws_need_seed(B, N, K);
    if (ctx->ws_bytes < need)
        return kb_fail(ctx, KB_ERR_WORKSPACE, "kb_seed_kmeanspp needs %zu bytes of workspace", need);
    SeedWs w;
    size_t zero_bytes = 0;
    seed_carve(ctx->ws, B, N, K, &w, &zero_bytes);
    const int G = seed_ctas(ctx, B, N);
    if (G > 1) KB_MEMSET(ctx, ctx->ws, 0, zero_bytes);
    const int rows_per = (N + G - 1) / G;
    for (int round = 0; round < K; ++round) {
        if (vec)
            kb_launch(seed_round_kernel<4>, dim3(G, B), SD_T, 0, ctx->stream, N, D, K, round, G, rows_per, z, rows, s_lo, s_hi,
                      w);
        else
            kb_launch(seed_round_kernel<1>, dim3(G, B), SD_T, 0, ctx->stream, N, D, K, round, G, rows_per, z, rows, s_lo, s_hi,
                      w);
        KB_LAUNCH_CHECK(ctx, "seed_round_kernel");
    }
    return KB_OK;
}

// ---- restarts: the run with the smallest inertia among n_init consecutive instances --------------------
namespace {
__global__ void best_restart_kernel(int G, int n_init, const float* __restrict__ inertia, int32_t* __restrict__ best) {
    kb_grid_dependency_wait();
    const int g = blockIdx.x * blockDim.x + threadIdx.x;
    if (g >= G) return;
    int arg = -1;
    float v = INFINITY;
    for (int r = 0; r < n_init; ++r) {
        const float x = inertia[(size_t)g * n_init + r];
        if (x != x) continue;                                    // NaN: never chosen
        if (arg < 0 || x < v) { v = x; arg = r; }
    }
    best[g] = arg;
}
}  // namespace

kb_status kb_launch_best_restart(kb_ctx* ctx, int G, int n_init, const float* inertia, int32_t* best) {
    if (G == 0) return KB_OK;
    kb_launch(best_restart_kernel, (G + 127) / 128, 128, 0, ctx->stream, G, n_init, inertia, best);
    KB_LAUNCH_CHECK(ctx, "best_restart_kernel");
    return KB_OK;
}
