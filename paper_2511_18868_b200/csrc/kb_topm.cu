// kb_select_top_m: the M arms with the largest per-arm index U(k, s) (the masked argmax of Sec. 3.4 taken M
// times, for generating M candidates per iteration).
//
// A value and its flat arm index pack into one 64-bit key (orderable fp32 bits, then the inverted index), so all
// keys of an instance are distinct and totally ordered: the j-th arm is simply the largest key BELOW the (j-1)-th.
// One launch per rank j: every CTA streams its slice once (float4 loads, four in flight), keeps the largest key
// under the previous winner, the CTAs of an instance meet in one atomicMax and the last one to finish writes
// the arm.  Exact (comparisons only), sorted output, no exclusion list; M passes over arm_index, meant for small M.
#include "kb_internal.cuh"

namespace {

constexpr int TM_T = 256;
constexpr int TM_U = 4;

struct TopWs {
    unsigned long long* key;   // [B][M]
    unsigned* done;            // [B][M]
};

__device__ __forceinline__ void top_take(float v, unsigned idx, unsigned long long limit, unsigned long long& best) {
    if (!(v > -INFINITY)) return;                                // pruned (-inf) or NaN
    const unsigned long long key = ((unsigned long long)kb_orderable(v) << 32) | (unsigned long long)(0xffffffffu - idx);
    if (key < limit && key > best) best = key;
}

template <bool VEC>
__global__ void __launch_bounds__(TM_T)
top_round_kernel(int NS, int M, int round, int G, int per, const float* __restrict__ arm_index, TopWs w,
                 int32_t* __restrict__ top_arm, float* __restrict__ top_val) {
    kb_grid_dependency_wait();
    __shared__ unsigned long long s_red[TM_T / 32];
    const int b = blockIdx.y, tid = threadIdx.x, lane = tid & 31;
    const size_t slot = (size_t)b * M + round;
    // the previous rank's key (final: its launch has completed); 0 there means nothing valid is left
    const unsigned long long limit = round == 0 ? ~0ull : w.key[slot - 1];
    unsigned long long best = 0ull;
    const float* v = arm_index + (size_t)b * NS;
    const int e0 = blockIdx.x * per, e1 = min(NS, e0 + per);
    if (limit != 0ull) {
        if (VEC) {
            const float4* v4 = reinterpret_cast<const float4*>(v);
            const int q1 = (e1 + 3) >> 2;                        // NS % 4 == 0 and per % 4 == 0 on this path
            for (int q = (e0 >> 2) + tid; q < q1; q += TM_T * TM_U) {
                float4 x[TM_U];
#pragma unroll
                for (int u = 0; u < TM_U; ++u)
                    x[u] = q + u * TM_T < q1 ? __ldg(v4 + q + u * TM_T) : make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
#pragma unroll
                for (int u = 0; u < TM_U; ++u) {
                    const unsigned i = (unsigned)(q + u * TM_T) << 2;
                    top_take(x[u].x, i, limit, best);
                    top_take(x[u].y, i + 1, limit, best);
                    top_take(x[u].z, i + 2, limit, best);
                    top_take(x[u].w, i + 3, limit, best);
                }
            }
        } else {
            for (int i = e0 + tid; i < e1; i += TM_T) top_take(__ldg(v + i), (unsigned)i, limit, best);
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const unsigned long long other = __shfl_xor_sync(0xffffffffu, best, o);
        best = other > best ? other : best;
    }
    if (lane == 0) s_red[tid >> 5] = best;
    __syncthreads();
    if (tid != 0) return;
#pragma unroll
    for (int i = 1; i < TM_T / 32; ++i) best = s_red[i] > best ? s_red[i] : best;
    if (G > 1) {
        if (best) atomicMax(&w.key[slot], best);
        __threadfence();
        if (atomicAdd(&w.done[slot], 1u) != (unsigned)G - 1u) return;
        __threadfence();
        best = atomicMax(&w.key[slot], 0ull);
    } else {
        w.key[slot] = best;                                      // the next rank reads it
    }
    if (best == 0ull) {
        top_arm[slot] = -1;
        if (top_val) top_val[slot] = -INFINITY;
    } else {
        top_arm[slot] = (int32_t)(0xffffffffu - (unsigned)(best & 0xffffffffull));
        if (top_val) top_val[slot] = kb_from_orderable((unsigned)(best >> 32));
    }
}

}  // namespace

size_t kb_ws_need_topm(int B, int M) {
    if (B < 1 || M < 1) return 0;
    return kb_align256((size_t)B * M * 8) + kb_align256((size_t)B * M * 4);
}

kb_status kb_launch_top_m(kb_ctx* ctx, int B, int NS, int M, const float* arm_index, int32_t* top_arm, float* top_val) {
    if (B == 0 || M == 0) return KB_OK;
    const size_t need = kb_ws_need_topm(B, M);
    if (ctx->ws_bytes < need)
        return kb_fail(ctx, KB_ERR_WORKSPACE, "kb_select_top_m needs %zu bytes of workspace", need);
    TopWs w;
    w.key = reinterpret_cast<unsigned long long*>(ctx->ws);
    w.done = reinterpret_cast<unsigned*>(ctx->ws + kb_align256((size_t)B * M * 8));
    KB_MEMSET(ctx, ctx->ws, 0, need);
    long want = (8L * ctx->sm_count + B - 1) / B;
    long cap = ((long)NS + TM_T * TM_U * 4 - 1) / (TM_T * TM_U * 4);
    long G = want < cap ? want : cap;
    if (G < 1) G = 1;
    int per = (int)((NS + G - 1) / G);
    per = (per + 3) & ~3;
    const bool vec = (NS % 4 == 0) && (((uintptr_t)arm_index & 15) == 0);
    for (int round = 0; round < M; ++round) {
        if (vec)
            kb_launch(top_round_kernel<true>, dim3((unsigned)G, B), TM_T, 0, ctx->stream, NS, M, round, (int)G, per, arm_index, w,
                      top_arm, top_val);
        else
            kb_launch(top_round_kernel<false>, dim3((unsigned)G, B), TM_T, 0, ctx->stream, NS, M, round, (int)G, per, arm_index, w,
                      top_arm, top_val);
        KB_LAUNCH_CHECK(ctx, "top_round_kernel");
    }
    return KB_OK;
}
