// kb_prune: roofline floor vs incumbent, saturation mask M_{i,s} (Sec. 3.4)
// and the gain bound B(k,s) of Assumption 1.  Keep bits are packed per candidate.
// Streaming: 12-16 bytes in and 4 bytes out per candidate, plus 4*S bytes when
// the bound is written.
//
// Vector path (S in {4, 8, 16, 32}): a thread owns four strategies of a row, so the
// bound leaves as float4 stores and the keep bits of a row are OR-ed across its
// S/4 lanes with shuffles.  Divisions would bind the kernel (three per arm), so a quotient whose
// divisor is fixed per thread is the product with the divisor's reciprocal; only where that leaves
// the floor within a few roundings of the incumbent is it redone with one fused residual correction,
// which gives the correctly rounded fp32 quotient for ordinary operands, so an arm whose floor
// equals the incumbent exactly is still pruned (strict <), as the definition says.  The bound is
// 1 - T_lb / T_k by one saturating multiply-add (absolute error below 3e-7).
// Generic path (any S <= 32): one thread per candidate, bound rows staged through
// shared memory so that they still leave the SM as full lines.
#include "kb_internal.cuh"

namespace {

constexpr int PR_T = 128;
constexpr int PV_T = 256;


__global__ void __launch_bounds__(PV_T)
prune_vec_kernel(int N, int S, int K, int R, int G, const float* __restrict__ flops, const float* __restrict__ bytes,
                 const float* __restrict__ peak_flops, const float* __restrict__ peak_bw,
                 const float* __restrict__ t_inc, const float* __restrict__ t_cur,
                 const int32_t* __restrict__ labels, const float* __restrict__ hsig,
                 const int32_t* __restrict__ target, float theta, uint32_t* __restrict__ keep,
                 uint32_t* __restrict__ kept, float* __restrict__ bound, int* __restrict__ dev_status) {
    kb_grid_dependency_wait();
    __shared__ unsigned s_kept[PV_T / 32];
    const int b = blockIdx.y, tid = threadIdx.x, lane = tid & 31;
    const int vps = S >> 2;                  // lanes per row: 1, 2, 4 or 8
    const int q = tid % vps;
    const int rstep = PV_T / vps;
    const bool sat = labels != nullptr;
    // per-strategy constants: the block forms the reciprocals once (a thread handles only a few rows, so eight
    // divisions of its own would cost as much as its share of the work)
    __shared__ float s_rP[32], s_rW[32];
    if (tid < S) {
        s_rP[tid] = 1.f / peak_flops[tid];
        s_rW[tid] = 1.f / peak_bw[tid];
    }
    __syncthreads();
    float P[4], W[4], rP[4], rW[4];
    int tg[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        P[i] = peak_flops[4 * q + i];
        W[i] = peak_bw[4 * q + i];
        rP[i] = s_rP[4 * q + i];
        rW[i] = s_rW[4 * q + i];
        int t = sat ? target[4 * q + i] : 0;
        if (t < 0 || t >= R) { if (sat) atomicOr(dev_status, 2); t = 0; }
        tg[i] = t;
    }
    const float tinc = t_inc[b];
    const int rows_per = (N + G - 1) / G;
    const int r0 = blockIdx.x * rows_per, r1 = min(N, r0 + rows_per);
    unsigned count = 0;
    constexpr int U = 4;                     // rows in flight per thread
    // the trip count is the same for every thread of the block, so the shuffles below are
    // always executed by full warps; rows past the end are computed on clamped inputs and dropped
    const int trips = (max(r1 - r0, 0) + U * rstep - 1) / (U * rstep);
    for (int it = 0; it < trips; ++it) {
        const int rb = r0 + tid / vps + it * U * rstep;
        float F[U], Q[U], Tk[U];
        int lab[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const size_t i = (size_t)b * N + min(rb + u * rstep, r1 - 1);   // clamped: loads stay in range
            F[u] = __ldg(flops + i);
            Q[u] = __ldg(bytes + i);
            Tk[u] = bound ? __ldg(t_cur + i) : 1.f;
            lab[u] = sat ? __ldg(labels + i) : 0;
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int r = rb + u * rstep;
            const bool live = r < r1;
            const size_t i = (size_t)b * N + min(r, r1 - 1);
            int lb_ = lab[u];
            if (sat && (lb_ < 0 || lb_ >= K)) { atomicOr(dev_status, 1); lb_ = 0; }
            const float* h = sat ? hsig + ((size_t)b * K + lb_) * R : nullptr;
            unsigned bits = 0;
            float g[4];
            const float rT = 1.f / Tk[u];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                // quotients by the reciprocal; where that leaves the floor within a few roundings of the incumbent
                // the decision is taken on the correctly rounded quotients (strict <: equality prunes)
                float tlb = fmaxf(F[u] * rP[k], Q[u] * rW[k]);
                if (fabsf(tlb - tinc) <= 2e-6f * tinc)
                    tlb = fmaxf(kb_div_by(F[u], P[k], rP[k]), kb_div_by(Q[u], W[k], rW[k]));
                bool ok = tlb < tinc;
                if (sat) ok = ok && (__ldg(h + tg[k]) < theta);
                if (ok) bits |= 1u << (4 * q + k);
                g[k] = __saturatef(fmaf(-tlb, rT, 1.f));     // clip(1 - T_lb / T_k, 0, 1); NaN (0/0) -> 0, as the definition does
            }
            for (int o = 1; o < vps; o <<= 1) bits |= __shfl_xor_sync(0xffffffffu, bits, o);
            if (live && q == 0) { keep[i] = bits; count += __popc(bits); }
            if (live && bound) *reinterpret_cast<float4*>(bound + i * S + 4 * q) = make_float4(g[0], g[1], g[2], g[3]);
        }
    }
    if (kept) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) count += __shfl_xor_sync(0xffffffffu, count, o);
        if (lane == 0) s_kept[tid >> 5] = count;
        __syncthreads();
        if (tid == 0) {
            unsigned tot = 0;
            for (int w = 0; w < PV_T / 32; ++w) tot += s_kept[w];
            if (tot) atomicAdd(&kept[b], tot);
        }
    }
}

__global__ void __launch_bounds__(PR_T)
prune_kernel(int N, int S, int K, int R, const float* __restrict__ flops, const float* __restrict__ bytes,
             const float* __restrict__ peak_flops, const float* __restrict__ peak_bw,
             const float* __restrict__ t_inc, const float* __restrict__ t_cur, const int32_t* __restrict__ labels,
             const float* __restrict__ hsig, const int32_t* __restrict__ target, float theta,
             uint32_t* __restrict__ keep, uint32_t* __restrict__ kept, float* __restrict__ bound,
             int* __restrict__ dev_status) {
    kb_grid_dependency_wait();
    extern __shared__ float tile[];  // [PR_T][S+1] when the bound is written
    __shared__ float sP[32], sW[32];
    __shared__ int sT[32];
    __shared__ unsigned s_kept;
    const int b = blockIdx.y, tid = threadIdx.x;
    const int r0 = blockIdx.x * PR_T;
    const int row = r0 + tid;
    const bool sat = labels != nullptr;
    if (tid < S) {
        sP[tid] = peak_flops[tid];
        sW[tid] = peak_bw[tid];
        int tg = sat ? target[tid] : 0;
        if (tg < 0 || tg >= R) { if (sat) atomicOr(dev_status, 2); tg = 0; }
        sT[tid] = tg;
    }
    if (tid == 0) s_kept = 0;
    __syncthreads();
    const float tinc = t_inc[b];
    uint32_t bits = 0;
    if (row < N) {
        const size_t i = (size_t)b * N + row;
        const float F = flops[i], Q = bytes[i];
        const float Tk = bound ? t_cur[i] : 1.f;
        const float* h = nullptr;
        if (sat) {
            int lab = labels[i];
            if (lab < 0 || lab >= K) { atomicOr(dev_status, 1); lab = 0; }
            h = hsig + ((size_t)b * K + lab) * R;
        }
        for (int s = 0; s < S; ++s) {
            float tlb = fmaxf(F / sP[s], Q / sW[s]);
            bool ok = tlb < tinc;
            if (sat) ok = ok && (__ldg(h + sT[s]) < theta);
            if (ok) bits |= (1u << s);
            if (bound) {
                float g = (Tk - tlb) / Tk;
                g = g > 0.f ? g : 0.f;  // also maps NaN (0/0) to 0, as the definition does
                g = g < 1.f ? g : 1.f;
                tile[tid * (S + 1) + s] = g;
            }
        }
        keep[i] = bits;
    }
    if (kept) {
        unsigned c = __popc(bits);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) c += __shfl_xor_sync(0xffffffffu, c, o);
        if ((tid & 31) == 0 && c) atomicAdd(&s_kept, c);
    }
    __syncthreads();
    if (kept && tid == 0 && s_kept) atomicAdd(&kept[b], s_kept);
    if (bound) {
        const int rows = min(PR_T, N - r0);
        float* dst = bound + ((size_t)b * N + r0) * S;
        for (int e = tid; e < rows * S; e += PR_T) {
            int r = e / S, s = e - r * S;
            dst[e] = tile[r * (S + 1) + s];
        }
    }
}

}  // namespace

kb_status kb_launch_prune(kb_ctx* ctx, int B, int N, int S, int K, int R, const float* flops, const float* bytes,
                          const float* peak_flops, const float* peak_bw, const float* t_inc, const float* t_cur,
                          const int32_t* labels, const float* hsig, const int32_t* target, float theta,
                          uint32_t* keep, uint32_t* kept, float* bound) {
    if (B == 0) return KB_OK;
    if (kept) {
        KB_MEMSET(ctx, kept, 0, (size_t)B * sizeof(uint32_t));
    }
    if (N == 0) return KB_OK;
    const bool vec = (S == 4 || S == 8 || S == 16 || S == 32) && (((uintptr_t)bound & 15) == 0);
    if (vec) {
        // one full wave: as many blocks as the device holds at once (the kernel's registers decide), split
        // over the instances; a grid of a wave and a fraction would run as long as two waves
        static int per_sm = 0;
        if (per_sm == 0) {
            int n = 0;
            if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, prune_vec_kernel, PV_T, 0) != cudaSuccess || n < 1) n = 2;
            per_sm = n;
        }
        long want = ((long)per_sm * ctx->sm_count) / B;
        if (want < 1) want = 1;
        long cap = ((long)N * (S / 4) + PV_T - 1) / PV_T;
        int G = (int)(want > cap ? cap : want);
        if (G < 1) G = 1;
        kb_launch(prune_vec_kernel, dim3(G, B), PV_T, 0, ctx->stream, N, S, K, R, G, flops, bytes, peak_flops, peak_bw, t_inc,
                                                             t_cur, labels, hsig, target, theta, keep, kept, bound,
                                                             ctx->dev_status);
        KB_LAUNCH_CHECK(ctx, "prune_vec_kernel");
        return KB_OK;
    }
    dim3 grid((N + PR_T - 1) / PR_T, B);
    size_t smem = bound ? (size_t)PR_T * (S + 1) * sizeof(float) : 0;
    kb_launch(prune_kernel, grid, PR_T, smem, ctx->stream, N, S, K, R, flops, bytes, peak_flops, peak_bw, t_inc, t_cur,
                                                    labels, hsig, target, theta, keep, kept, bound,
                                                    ctx->dev_status);
    KB_LAUNCH_CHECK(ctx, "prune_kernel");
    return KB_OK;
}
