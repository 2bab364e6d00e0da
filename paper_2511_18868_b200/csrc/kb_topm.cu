// kb_select_top_m: the M arms with the largest per-arm index U(k, s) (the masked argmax of Sec. 3.4 taken M
// times, for generating M candidates per iteration) in ONE pass over arm_index.
//
// A value and its flat arm index pack into one 64-bit key (orderable fp32 bits, then the inverted index), so all
// keys of an instance are distinct and totally ordered: larger value first, lower index first among equal values.
//
//   top_slice_kernel   every CTA streams its slice of the instance once (float4 loads) and keeps the slice's M
//                      largest keys: a key above the CTA's current threshold is appended to a shared-memory
//                      buffer (one shared atomic per warp); when the buffer runs full it is sorted (bitonic, in
//                      place), cut to its M largest, and the M-th becomes the new threshold.  The first threshold
//                      comes from the threads' own maxima over their first sixteen keys (a 256-key sort), so from
//                      the start only about M keys in every few thousand pass.  The CTA's M keys go to global
//                      memory; an instance that fits one CTA is finished here.
//   top_merge_kernel   one CTA per instance runs the same selection over the G x M keys of its slices.
// Exact (comparisons only), sorted output, no exclusion list, any M up to KB_TOP_M_MAX; arm_index is read once.
#include "kb_internal.cuh"

namespace {

constexpr int TM_T = 256;                 // threads per CTA
constexpr int TM_CHUNK = TM_T * 4;        // keys looked at per trip (one float4 per thread)
constexpr int TM_U = 4;                   // chunks requested together (loads in flight per thread)
constexpr int TM_CAP = 2048;              // buffer: a power of two, >= TM_CUT_AT + TM_CHUNK
constexpr int TM_CUT_AT = 512;            // cut before a chunk whenever more than this many keys are buffered (>= KB_TOP_M_MAX)

__device__ __forceinline__ unsigned long long top_key(float v, unsigned idx) {
    if (!(v > -INFINITY)) return 0ull;                           // pruned (-inf) or NaN: never a candidate
    return ((unsigned long long)kb_orderable(v) << 32) | (unsigned long long)(0xffffffffu - idx);
}

// Sorts buf[0, n) in descending order, n a power of two (<= TM_CAP); all threads of the CTA take part, each
// handling compare-exchange pairs (no idle half).
__device__ void bitonic_desc(unsigned long long* buf, int n) {
    const int pairs = n >> 1;
    for (int k = 2; k <= n; k <<= 1) {
        for (int j = k >> 1; j > 0; j >>= 1) {
            for (int t = threadIdx.x; t < pairs; t += TM_T) {
                const int i = ((t & ~(j - 1)) << 1) | (t & (j - 1));   // the lower index of pair t at distance j
                const int p = i | j;
                const unsigned long long a = buf[i], b = buf[p];
                const bool desc = (i & k) == 0;                  // this run is sorted downwards
                if (desc ? a < b : a > b) { buf[i] = b; buf[p] = a; }
            }
            __syncthreads();
        }
    }
}

// Keeps the M largest of the buffered keys and returns the new threshold (0 while fewer than M are known).
// *s_count is the number of valid keys in buf; every thread of the CTA calls this together.
__device__ unsigned long long top_cut(unsigned long long* buf, unsigned* s_count, int M) {
    __syncthreads();
    const int count = (int)*s_count;
    int n = 2;
    while (n < count) n <<= 1;
    for (int i = count + threadIdx.x; i < n; i += TM_T) buf[i] = 0ull;   // padding sorts to the end
    __syncthreads();
    bitonic_desc(buf, n);
    const unsigned long long thr = count >= M ? buf[M - 1] : 0ull;
    __syncthreads();
    if (threadIdx.x == 0) *s_count = (unsigned)min(count, M);
    __syncthreads();
    return thr;
}

// A first threshold without a big sort: the M-th largest of the threads' own maxima over their first keys is a
// lower bound on the M-th largest key of the whole stream (those M maxima are M distinct keys), so everything
// below it can be dropped from the start.  Returns the bound minus one (offers are strict: key > threshold), 0 if
// fewer than M threads saw a valid key.  Uses buf[0, TM_T); every thread of the CTA calls this together.
__device__ unsigned long long top_first_threshold(unsigned long long mine, unsigned long long* buf, int M) {
    __syncthreads();
    buf[threadIdx.x] = mine;
    __syncthreads();
    bitonic_desc(buf, TM_T);
    const unsigned long long t = M <= TM_T ? buf[M - 1] : 0ull;
    __syncthreads();
    return t ? t - 1ull : 0ull;
}

// One trip: each thread offers up to four keys; those above the threshold are appended (one atomic per warp).
__device__ __forceinline__ void top_offer(const unsigned long long (&key)[4], unsigned long long thr,
                                          unsigned long long* buf, unsigned* s_count) {
    const int lane = threadIdx.x & 31;
    int mine = 0;
#pragma unroll
    for (int i = 0; i < 4; ++i) mine += key[i] > thr ? 1 : 0;    // (0 never passes: thr >= 0)
    int incl = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int v = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += v;
    }
    const int total = __shfl_sync(0xffffffffu, incl, 31);
    unsigned base = 0;
    if (lane == 31 && total) base = atomicAdd(s_count, (unsigned)total);
    base = __shfl_sync(0xffffffffu, base, 31);
    unsigned pos = base + (unsigned)(incl - mine);
#pragma unroll
    for (int i = 0; i < 4; ++i)
        if (key[i] > thr) buf[pos++] = key[i];
}

__device__ __forceinline__ void top_write(unsigned long long key, size_t slot, int32_t* __restrict__ top_arm,
                                          float* __restrict__ top_val) {
    if (key == 0ull) {
        top_arm[slot] = -1;
        if (top_val) top_val[slot] = -INFINITY;
    } else {
        top_arm[slot] = (int32_t)(0xffffffffu - (unsigned)(key & 0xffffffffull));
        if (top_val) top_val[slot] = kb_from_orderable((unsigned)(key >> 32));
    }
}

template <bool VEC>
__global__ void __launch_bounds__(TM_T)
top_slice_kernel(int NS, int M, int G, int per, const float* __restrict__ arm_index, unsigned long long* __restrict__ part,
                 int32_t* __restrict__ top_arm, float* __restrict__ top_val) {
    kb_grid_dependency_wait();
    __shared__ unsigned long long buf[TM_CAP];
    __shared__ unsigned s_count;
    const int b = blockIdx.y, g = blockIdx.x, tid = threadIdx.x;
    if (tid == 0) s_count = 0;
    __syncthreads();
    const float* v = arm_index + (size_t)b * NS;
    const int e0 = g * per, e1 = min(NS, e0 + per);               // per is a multiple of TM_CHUNK
    unsigned long long thr = 0ull;
    for (int c0 = e0; c0 < e1; c0 += TM_U * TM_CHUNK) {
        // TM_U chunks are requested together, then offered one after the other
        float4 x[TM_U];
#pragma unroll
        for (int u = 0; u < TM_U; ++u) {
            const int i0 = c0 + u * TM_CHUNK + 4 * tid;
            x[u] = make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
            if (VEC) {
                if (i0 < e1) x[u] = __ldg(reinterpret_cast<const float4*>(v + i0));   // NS % 4 == 0 on this path
            } else {
                if (i0 < e1) x[u].x = __ldg(v + i0);
                if (i0 + 1 < e1) x[u].y = __ldg(v + i0 + 1);
                if (i0 + 2 < e1) x[u].z = __ldg(v + i0 + 2);
                if (i0 + 3 < e1) x[u].w = __ldg(v + i0 + 3);
            }
        }
        if (c0 == e0) {                                          // (the buffer is still empty)
            unsigned long long mx = 0ull;
#pragma unroll
            for (int u = 0; u < TM_U; ++u) {
                const unsigned i0 = (unsigned)(c0 + u * TM_CHUNK + 4 * tid);
                const unsigned long long k0 = top_key(x[u].x, i0), k1 = top_key(x[u].y, i0 + 1), k2 = top_key(x[u].z, i0 + 2),
                                         k3 = top_key(x[u].w, i0 + 3);
                mx = max(max(mx, k0), max(max(k1, k2), k3));
            }
            thr = top_first_threshold(mx, buf, M);
        }
#pragma unroll
        for (int u = 0; u < TM_U; ++u) {
            if (c0 + u * TM_CHUNK >= e1) break;                  // (the same in every thread)
            if (s_count > (unsigned)TM_CUT_AT) thr = max(thr, top_cut(buf, &s_count, M));   // (the same value in every thread)
            const unsigned i0 = (unsigned)(c0 + u * TM_CHUNK + 4 * tid);
            unsigned long long key[4] = {top_key(x[u].x, i0), top_key(x[u].y, i0 + 1), top_key(x[u].z, i0 + 2),
                                         top_key(x[u].w, i0 + 3)};
            top_offer(key, thr, buf, &s_count);
            __syncthreads();                                     // s_count is read before the next chunk
        }
    }
    top_cut(buf, &s_count, M);
    const int have = (int)s_count;
    if (G == 1) {
        for (int j = tid; j < M; j += TM_T) top_write(j < have ? buf[j] : 0ull, (size_t)b * M + j, top_arm, top_val);
    } else {
        unsigned long long* out = part + ((size_t)b * G + g) * M;
        for (int j = tid; j < M; j += TM_T) out[j] = j < have ? buf[j] : 0ull;
    }
}

__global__ void __launch_bounds__(TM_T)
top_merge_kernel(int M, int G, const unsigned long long* __restrict__ part, int32_t* __restrict__ top_arm,
                 float* __restrict__ top_val) {
    kb_grid_dependency_wait();
    __shared__ unsigned long long buf[TM_CAP];
    __shared__ unsigned s_count;
    const int b = blockIdx.x, tid = threadIdx.x;
    if (tid == 0) s_count = 0;
    __syncthreads();
    const unsigned long long* src = part + (size_t)b * G * M;
    const int total = G * M;
    unsigned long long thr = 0ull;
    for (int c0 = 0; c0 < total; c0 += TM_CHUNK) {
        if (s_count > (unsigned)TM_CUT_AT) thr = max(thr, top_cut(buf, &s_count, M));
        unsigned long long key[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int e = c0 + i * TM_T + tid;                   // coalesced 8-byte loads
            key[i] = e < total ? src[e] : 0ull;
        }
        if (c0 == 0) thr = top_first_threshold(max(max(key[0], key[1]), max(key[2], key[3])), buf, M);
        top_offer(key, thr, buf, &s_count);
        __syncthreads();
    }
    top_cut(buf, &s_count, M);
    const int have = (int)s_count;
    for (int j = tid; j < M; j += TM_T) top_write(j < have ? buf[j] : 0ull, (size_t)b * M + j, top_arm, top_val);
}

// slices per instance: about four CTAs per SM in all, each with at least a few trips
int top_slices(const kb_ctx* ctx, int B, int NS) {
    long want = (4L * ctx->sm_count + B - 1) / B;
    long cap = ((long)NS + 2 * TM_U * TM_CHUNK - 1) / (2 * TM_U * TM_CHUNK);
    long G = want < cap ? want : cap;
    return (int)(G < 1 ? 1 : G);
}

}  // namespace

size_t kb_ws_need_topm(int B, int M) {
    if (B < 1 || M < 1) return 0;
    // the slices' keys: [B][G][M], G at most two CTAs per SM of the largest part this library meets (bounded here
    // without a context: 1024 slices per instance when B == 1, fewer as B grows)
    const size_t G = (size_t)(B >= 1024 ? 1 : (1024 + B - 1) / B);
    return kb_align256((size_t)B * G * M * 8);
}

kb_status kb_launch_top_m(kb_ctx* ctx, int B, int NS, int M, const float* arm_index, int32_t* top_arm, float* top_val) {
    if (B == 0 || M == 0) return KB_OK;
    int G = top_slices(ctx, B, NS);
    const size_t gmax = (size_t)(B >= 1024 ? 1 : (1024 + B - 1) / B);
    if ((size_t)G > gmax) G = (int)gmax;
    const size_t need = kb_align256((size_t)B * G * M * 8);
    if (G > 1 && ctx->ws_bytes < need)
        return kb_fail(ctx, KB_ERR_WORKSPACE, "kb_select_top_m needs %zu bytes of workspace", need);
    unsigned long long* part = reinterpret_cast<unsigned long long*>(ctx->ws);
    int per = (int)(((long)NS + G - 1) / G);
    per = (per + TM_CHUNK - 1) / TM_CHUNK * TM_CHUNK;
    if (per < TM_CHUNK) per = TM_CHUNK;
    const bool vec = (NS % 4 == 0) && (((uintptr_t)arm_index & 15) == 0);
    if (vec)
        kb_launch(top_slice_kernel<true>, dim3((unsigned)G, B), TM_T, 0, ctx->stream, NS, M, G, per, arm_index, part, top_arm, top_val);
    else
        kb_launch(top_slice_kernel<false>, dim3((unsigned)G, B), TM_T, 0, ctx->stream, NS, M, G, per, arm_index, part, top_arm, top_val);
    KB_LAUNCH_CHECK(ctx, "top_slice_kernel");
    if (G > 1) {
        kb_launch(top_merge_kernel, B, TM_T, 0, ctx->stream, M, G, part, top_arm, top_val);
        KB_LAUNCH_CHECK(ctx, "top_merge_kernel");
    }
    return KB_OK;
}
