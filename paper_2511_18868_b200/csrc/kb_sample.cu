// kb_sample_member: the within-cluster draw of k_t (Sec. 3.4, "Action selection"; Algorithm 1,
// "Sample k_t in C_{I_t}").
//
// Once the pair (I_t, S_t) is chosen, k_t is drawn from the members of cluster I_t with
// P(k) proportional to exp(V_hw(k, S_t)), V_hw(k, s) = theta_sat - h(k)[Target(s)].  The draw is a
// segmented Gumbel-max: every member gets V_hw + G with G = -ln(-ln u), u uniform in (0, 1), and the
// largest perturbed value wins (lowest index on ties), which samples exactly that softmax with one
// pass, no normalising sum and no second pass for a prefix search.  u comes from a counter-based
// generator (Philox4x32, 10 rounds) keyed by the caller's seed and addressed by
// (candidate, instance, t[b], 0), so the draw does not depend on how the rows are spread over
// threads and a replay with the same seed and step counter repeats it.
//
// Traffic: labels once (4 bytes per candidate) plus one 32-byte sector of h_cand per member of the
// chosen cluster.  One kernel: every CTA reduces its rows to a packed 64-bit key (perturbed value,
// then lowest index), the CTAs of an instance meet in one atomicMax, and the last CTA of the
// instance to finish unpacks the result.  An instance that fits one CTA skips the atomics.
#include "kb_internal.cuh"

namespace {

constexpr int SM_T = 256;      // threads per CTA
constexpr int SM_U = 4;        // label loads in flight per thread
constexpr int SM_ROWS = SM_T * SM_U * 4;   // rows per CTA at least (when the instance is split): one vector trip

struct SampleWs {
    unsigned long long* key;   // [B] packed (perturbed value, inverted row)
    unsigned* done;            // [B] CTAs of the instance that have finished
};

__device__ __forceinline__ void sample_store(unsigned long long key, int32_t* member, float* member_val, int b) {
    if (key == 0ull) {
        member[b] = -1;
        if (member_val) member_val[b] = -INFINITY;
    } else {
        member[b] = (int32_t)(0xffffffffu - (unsigned)(key & 0xffffffffull));
        if (member_val) member_val[b] = kb_from_orderable((unsigned)(key >> 32));
    }
}

template <bool VEC>
__global__ void __launch_bounds__(SM_T)
sample_member_kernel(int N, int K, int S, int R, int rows_per, int G, const int32_t* __restrict__ labels,
                     const int32_t* __restrict__ cluster_arm, const float* __restrict__ h_cand,
                     const int32_t* __restrict__ target, float theta, uint32_t seed_lo, uint32_t seed_hi,
                     const int32_t* __restrict__ t, SampleWs w, int32_t* __restrict__ member,
                     float* __restrict__ member_val, int* __restrict__ dev_status) {
    kb_grid_dependency_wait();
    __shared__ unsigned long long s_red[SM_T / 32];
    const int b = blockIdx.y, tid = threadIdx.x, lane = tid & 31;
    const int ca = cluster_arm[b];
    unsigned long long best = 0ull;
    bool draw = ca >= 0;
    int I = 0, col = 0;
    if (draw) {
        if (ca >= K * S) {
            if (tid == 0) atomicOr(dev_status, 4);
            draw = false;
        } else {
            I = ca / S;
            col = target[ca - I * S];
            if (col < 0 || col >= R) {
                if (tid == 0) atomicOr(dev_status, 2);
                draw = false;
            }
        }
    }
    if (draw) {
        const int r0 = blockIdx.x * rows_per, r1 = min(N, r0 + rows_per);
        const int32_t* lb = labels + (size_t)b * N;
        const float* hb = h_cand + (size_t)b * N * R + col;
        const uint32_t tb = (uint32_t)t[b];
        // one candidate of the chosen cluster: signature entry, uniform, perturbed value, packed key
        auto take = [&](int r) {
            const float h = __ldg(hb + (size_t)r * R);
            const uint32_t w0 = kb_philox4x32_10_word0((uint32_t)r, (uint32_t)b, tb, 0u, seed_lo, seed_hi);
            const float uni = ((float)(w0 >> 9) + 0.5f) * (1.0f / 8388608.0f);   // 23 bits: exact
            const float v = (theta - h) - logf(-logf(uni));
            if (!(v > -INFINITY)) return;                                        // NaN or -inf: never drawn
            const unsigned long long key =
                ((unsigned long long)kb_orderable(v) << 32) | (unsigned long long)(0xffffffffu - (unsigned)r);
            best = key > best ? key : best;
        };
        if (VEC) {
            // r0 is a multiple of 4 (the host rounds rows_per up): 16 labels per thread and trip, four loads in flight
            const int4* lb4 = reinterpret_cast<const int4*>(lb);
            const int q1 = (r1 + 3) >> 2;                      // N % 4 == 0 on this path, so whole quads only
            for (int q = (r0 >> 2) + tid; q < q1; q += SM_T * SM_U) {
                int4 lab[SM_U];
#pragma unroll
                for (int u = 0; u < SM_U; ++u)
                    lab[u] = q + u * SM_T < q1 ? __ldg(lb4 + q + u * SM_T) : make_int4(-1, -1, -1, -1);
#pragma unroll
                for (int u = 0; u < SM_U; ++u) {
                    const int r = (q + u * SM_T) << 2;
                    if (lab[u].x == I) take(r);
                    if (lab[u].y == I) take(r + 1);
                    if (lab[u].z == I) take(r + 2);
                    if (lab[u].w == I) take(r + 3);
                }
            }
        } else {
            for (int base = r0 + tid; base < r1; base += SM_T * SM_U) {
                int lab[SM_U];
#pragma unroll
                for (int u = 0; u < SM_U; ++u) {
                    const int r = base + u * SM_T;
                    lab[u] = r < r1 ? __ldg(lb + r) : -1;
                }
#pragma unroll
                for (int u = 0; u < SM_U; ++u)
                    if (lab[u] == I) take(base + u * SM_T);
            }
        }
    }
    // block maximum
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const unsigned long long other = __shfl_xor_sync(0xffffffffu, best, o);
        best = other > best ? other : best;
    }
    if (lane == 0) s_red[tid >> 5] = best;
    __syncthreads();
    if (tid != 0) return;
#pragma unroll
    for (int i = 1; i < SM_T / 32; ++i) best = s_red[i] > best ? s_red[i] : best;
    if (G == 1) {
        sample_store(best, member, member_val, b);
        return;
    }
    if (best) atomicMax(&w.key[b], best);
    __threadfence();
    const unsigned ticket = atomicAdd(&w.done[b], 1u);
    if (ticket == (unsigned)G - 1u) {
        __threadfence();
        sample_store(atomicMax(&w.key[b], 0ull), member, member_val, b);
    }
}

int sample_ctas(const kb_ctx* ctx, int B, int N) {
    long want = (8L * ctx->sm_count + B - 1) / B;      // eight CTAs of 256 threads fit an SM
    long cap = ((long)N + SM_ROWS - 1) / SM_ROWS;
    long g = want < cap ? want : cap;
    return (int)(g < 1 ? 1 : g);
}

}  // namespace

size_t kb_ws_need_sample(int B) { return 2 * kb_align256((size_t)(B > 0 ? B : 1) * 8); }

kb_status kb_launch_sample_member(kb_ctx* ctx, int B, int N, int K, int S, int R, const int32_t* labels,
                                  const int32_t* cluster_arm, const float* h_cand, const int32_t* target,
                                  float theta_sat, uint64_t seed, const int32_t* t, int32_t* member,
                                  float* member_val) {
    if (B == 0) return KB_OK;
    const int G = sample_ctas(ctx, B, N);
    SampleWs w{nullptr, nullptr};
    if (G > 1) {
        const size_t need = kb_ws_need_sample(B);
        if (ctx->ws_bytes < need)
            return kb_fail(ctx, KB_ERR_WORKSPACE, "kb_sample_member needs %zu bytes of workspace", need);
        w.key = reinterpret_cast<unsigned long long*>(ctx->ws);
        w.done = reinterpret_cast<unsigned*>(ctx->ws + kb_align256((size_t)B * 8));
        KB_MEMSET(ctx, ctx->ws, 0, need);
    }
    const bool vec = (N % 4 == 0) && (((uintptr_t)labels & 15) == 0);
    int rows_per = (N + G - 1) / G;
    rows_per = (rows_per + 3) & ~3;                    // every CTA starts on a quad of labels
    const uint32_t s_lo = (uint32_t)(seed & 0xffffffffu), s_hi = (uint32_t)(seed >> 32);
    if (vec)
        kb_launch(sample_member_kernel<true>, dim3(G, B), SM_T, 0, ctx->stream, N, K, S, R, rows_per, G, labels, cluster_arm,
                  h_cand, target, theta_sat, s_lo, s_hi, t, w, member, member_val, ctx->dev_status);
    else
        kb_launch(sample_member_kernel<false>, dim3(G, B), SM_T, 0, ctx->stream, N, K, S, R, rows_per, G, labels, cluster_arm,
                  h_cand, target, theta_sat, s_lo, s_hi, t, w, member, member_val, ctx->dev_status);
    KB_LAUNCH_CHECK(ctx, "sample_member_kernel");
    return KB_OK;
}
