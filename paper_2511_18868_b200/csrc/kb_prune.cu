// kb_prune: roofline floor vs incumbent, saturation mask M_{i,s} (Sec. 3.4)
// and the gain bound B(k,s) of Assumption 1, one thread per candidate, keep
// bits packed per candidate.  Streaming: 12-16 bytes in and 4 bytes out per
// candidate, plus 4*S bytes when the bound is written (staged through shared
// memory so that the [N][S] rows leave the SM as full 128-byte lines).
#include "kb_internal.cuh"

namespace {

constexpr int PR_T = 128;

__global__ void __launch_bounds__(PR_T)
prune_kernel(int N, int S, int K, int R, const float* __restrict__ flops, const float* __restrict__ bytes,
             const float* __restrict__ peak_flops, const float* __restrict__ peak_bw,
             const float* __restrict__ t_inc, const float* __restrict__ t_cur, const int32_t* __restrict__ labels,
             const float* __restrict__ hsig, const int32_t* __restrict__ target, float theta,
             uint32_t* __restrict__ keep, uint32_t* __restrict__ kept, float* __restrict__ bound,
             int* __restrict__ dev_status) {
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
    dim3 grid((N + PR_T - 1) / PR_T, B);
    size_t smem = bound ? (size_t)PR_T * (S + 1) * sizeof(float) : 0;
    prune_kernel<<<grid, PR_T, smem, ctx->stream>>>(N, S, K, R, flops, bytes, peak_flops, peak_bw, t_inc, t_cur,
                                                    labels, hsig, target, theta, keep, kept, bound,
                                                    ctx->dev_status);
    KB_LAUNCH_CHECK(ctx, "prune_kernel");
    return KB_OK;
}
