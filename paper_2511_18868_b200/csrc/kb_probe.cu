// kb_probe_peaks: the two arithmetic ceilings the benchmark divides by, measured on the device
// the context is bound to, in the instruction shapes the library's kernels use.
//
//   fp32 FMA      every resident thread runs independent register-resident FFMA chains
//                 (the ceiling of the row-wise assign and of the fused / cooperative fits);
//   tensor cores  one CTA per SM issues back-to-back tcgen05.mma, M = 128, N = 128, A from
//                 tensor memory, B by shared-memory descriptor (128-byte swizzle, K-major), fp32
//                 accumulation -- kind::f16 (K = 16 per instruction) and kind::tf32 (K = 8), the two
//                 splits of the tensor-core assign.  The products are never read: the rate does not
//                 depend on the operand values.
// Each figure is work / CUDA-event time of one launch that runs for about a millisecond.
#include <string.h>

#include "kb_internal.cuh"

namespace {

constexpr int FF_CHAINS = 16;      // independent FMA chains per thread
constexpr int FF_THREADS = 512;
constexpr int FF_CTAS_PER_SM = 4;

__global__ void __launch_bounds__(FF_THREADS) probe_ffma_kernel(int iters, float seed, int* __restrict__ sink) {
    float a[FF_CHAINS];
#pragma unroll
    for (int i = 0; i < FF_CHAINS; ++i) a[i] = seed + (float)(threadIdx.x + i);
    const float m = 1.0f - seed * 1e-7f, c = seed * 1e-3f;
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int i = 0; i < FF_CHAINS; ++i) a[i] = fmaf(a[i], m, c);
    }
    float s = 0.f;
#pragma unroll
    for (int i = 0; i < FF_CHAINS; ++i) s += a[i];
    if (s == -12345.678f) atomicAdd(sink, 1);          // never true: keeps the chains alive
}

__device__ __forceinline__ uint32_t pr_smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
// K-major operand tile of 128-byte rows, 128-byte swizzle, 8-row groups 1024 bytes apart
__device__ __forceinline__ uint64_t pr_desc_sw128(uint32_t addr) {
    uint64_t d = (uint64_t)((addr & 0x3FFFFu) >> 4);
    d |= (uint64_t)1 << 16;
    d |= (uint64_t)(1024 >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}
__device__ __forceinline__ bool pr_mbar_try(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}

constexpr int PM_N = 128;                                   // accumulator tile: 128 x 128 fp32
constexpr uint32_t PM_IDESC_F16 = (1u << 4) | ((uint32_t)(PM_N >> 3) << 17) | (8u << 24);
constexpr uint32_t PM_IDESC_TF32 = (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(PM_N >> 3) << 17) | (8u << 24);
constexpr uint32_t PM_WAIT_LIMIT = 1u << 24;                // polls of the one bounded wait (well under a second)
constexpr int PM_SMEM = 128 * 1024;                         // one B tile (16 KB) is used; the size keeps one CTA per SM

// One product D[tmem] (+)= A[tmem] * B[smem descriptor]; `acc` == 0 overwrites the accumulator.
template <bool TF32>
__device__ __forceinline__ void pr_mma(uint32_t d, uint32_t a, uint64_t bdesc, uint32_t acc) {
    if (TF32) {
        asm volatile(
            "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
            "tcgen05.mma.cta_group::1.kind::tf32 [%0], [%1], %2, %3, p;\n\t}" ::"r"(d), "r"(a), "l"(bdesc),
            "r"(PM_IDESC_TF32), "r"(acc)
            : "memory");
    } else {
        asm volatile(
            "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
            "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}" ::"r"(d), "r"(a), "l"(bdesc),
            "r"(PM_IDESC_F16), "r"(acc)
            : "memory");
    }
}

// Two accumulators take turns, 16 products each (the first of a run overwrites), as the assign kernel's tiles do.
// The issuing loop is unrolled by 16 with every operand address a constant offset, so that what is timed is the
// tensor pipe and not the issuing thread's own address arithmetic (a lone warp runs its dependent integer
// instructions at a few cycles each: twenty of them per product would cost more than the product).
template <bool TF32>
__global__ void __launch_bounds__(128, 1) probe_mma_kernel(int iters, int* __restrict__ fail, long long* __restrict__ stamps) {
    extern __shared__ unsigned char pm_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>(((uintptr_t)pm_raw + 1023) & ~(uintptr_t)1023);
    __shared__ uint64_t bar;
    __shared__ uint32_t slot;
    const int tid = threadIdx.x, warp = tid >> 5;
    if (tid == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(pr_smem_u32(&bar)));
        asm volatile("fence.mbarrier_init.release.cluster;");
    }
    for (int i = tid; i < 16 * 1024 / 4; i += 128) reinterpret_cast<uint32_t*>(smem)[i] = 0u;
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(pr_smem_u32(&slot)) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;");
    }
    asm volatile("tcgen05.fence::before_thread_sync;");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    const uint32_t tmem = slot;
    // tensor memory: columns [0, 256) two accumulators, [256, 512) the A operand (its contents are whatever the
    // allocation held: any bit pattern multiplies at the same rate, and the products are never read)
    if (warp == 1) {
        // one elected lane of a converged warp issues, as in the assign kernel
        const uint64_t bdesc = pr_desc_sw128(pr_smem_u32(smem));
        uint32_t elected;
        asm volatile("{\n\t.reg .pred P;\n\telect.sync _|P, 0xffffffff;\n\tselp.u32 %0, 1, 0, P;\n\t}" : "=r"(elected));
        const long long c0 = clock64();
        unsigned long long n0;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(n0));
        if (elected) {
            for (int i = 0; i < iters; i += 16) {
                const uint32_t d = tmem + (uint32_t)((i >> 4) & 1) * 128u;
#pragma unroll
                for (int u = 0; u < 16; ++u)                           // 32-byte k-steps inside the swizzled row
                    pr_mma<TF32>(d, tmem + 256u + (uint32_t)u * 8u, bdesc + (uint64_t)((u & 3) * 2), u == 0 ? 0u : 1u);
            }
        }
        __syncwarp();
        if ((tid & 31) == 0) {
            asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(pr_smem_u32(&bar))
                         : "memory");
            bool ok = false;
            for (uint32_t i = 0; i < PM_WAIT_LIMIT && !ok; ++i) ok = pr_mbar_try(pr_smem_u32(&bar), 0u);
            if (!ok) atomicAdd(fail, 1);                              // the products did not retire in time: no figure
            if (blockIdx.x == 0) {                                    // SM cycles and nanoseconds of the whole stream
                unsigned long long n1;
                asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(n1));
                stamps[0] = clock64() - c0;
                stamps[1] = (long long)(n1 - n0);
            }
        }
        __syncwarp();
    }
    asm volatile("tcgen05.fence::before_thread_sync;");
    __syncthreads();
    if (warp == 0) {
        asm volatile("tcgen05.fence::after_thread_sync;");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem) : "memory");
    }
}

}  // namespace

extern "C" kb_status kb_probe_peaks(kb_ctx* ctx, kb_peak_probe* out) {
    if (!ctx || !out) return KB_ERR_INVALID_ARG;
    memset(out, 0, sizeof(*out));
    cudaEvent_t e0, e1;
    KB_CUDA(ctx, cudaEventCreate(&e0));
    KB_CUDA(ctx, cudaEventCreate(&e1));
    int* sink = ctx->dev_status + 16;                    // spare words behind the status word (256 bytes are owned)
    long long* stamps = reinterpret_cast<long long*>(ctx->dev_status + 32);   // [kind][cycles, ns], 8-byte aligned
    cudaStream_t st = ctx->stream;
    kb_status s = KB_OK;
    auto elapsed = [&](float* ms) -> bool {
        return cudaEventSynchronize(e1) == cudaSuccess && cudaEventElapsedTime(ms, e0, e1) == cudaSuccess;
    };
    do {
        if (cudaMemsetAsync(sink, 0, 2 * sizeof(int), st) != cudaSuccess ||
            cudaMemsetAsync(stamps, 0, 4 * sizeof(long long), st) != cudaSuccess) { s = KB_ERR_CUDA; break; }
        // ---- fp32 FMA: warm-up launch, then the timed one
        const int ff_iters = 4096, ff_grid = ctx->sm_count * FF_CTAS_PER_SM;
        float ms = 0.f;
        for (int rep = 0; rep < 2; ++rep) {
            cudaEventRecord(e0, st);
            probe_ffma_kernel<<<ff_grid, FF_THREADS, 0, st>>>(ff_iters, 1.0f, sink);
            cudaEventRecord(e1, st);
            if (cudaGetLastError() != cudaSuccess || !elapsed(&ms)) { s = KB_ERR_CUDA; break; }
        }
        if (s != KB_OK) break;
        out->ffma_ms = ms;
        out->ffma_tflops = 2.0 * (double)ff_grid * FF_THREADS * FF_CHAINS * ff_iters / (ms * 1e-3) / 1e12;
        // ---- tensor cores, both kinds
        if (cudaFuncSetAttribute(probe_mma_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, PM_SMEM) != cudaSuccess ||
            cudaFuncSetAttribute(probe_mma_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, PM_SMEM) != cudaSuccess) {
            s = KB_ERR_CUDA;
            break;
        }
        const int mm_iters = 16384;
        for (int tf32 = 0; tf32 < 2 && s == KB_OK; ++tf32) {
            for (int rep = 0; rep < 2; ++rep) {
                cudaEventRecord(e0, st);
                if (tf32) probe_mma_kernel<true><<<ctx->sm_count, 128, PM_SMEM, st>>>(mm_iters, sink + 1, stamps + 2);
                else probe_mma_kernel<false><<<ctx->sm_count, 128, PM_SMEM, st>>>(mm_iters, sink + 1, stamps);
                cudaEventRecord(e1, st);
                if (cudaGetLastError() != cudaSuccess || !elapsed(&ms)) { s = KB_ERR_CUDA; break; }
            }
            if (s != KB_OK) break;
            const double flops = 2.0 * 128.0 * PM_N * (tf32 ? 8.0 : 16.0) * mm_iters * ctx->sm_count;
            (tf32 ? out->mma_tf32_ms : out->mma_f16_ms) = ms;
            (tf32 ? out->mma_tf32_tflops : out->mma_f16_tflops) = flops / (ms * 1e-3) / 1e12;
        }
        if (s != KB_OK) break;
        int host[2] = {0, 0};
        long long hst[4] = {0, 0, 0, 0};
        if (cudaMemcpyAsync(host, sink, sizeof(host), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
            cudaMemcpyAsync(hst, stamps, sizeof(hst), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
            cudaStreamSynchronize(st) != cudaSuccess) { s = KB_ERR_CUDA; break; }
        out->mma_f16_cycles_per_instr = (float)((double)hst[0] / mm_iters);
        out->mma_tf32_cycles_per_instr = (float)((double)hst[2] / mm_iters);
        out->mma_f16_sm_mhz = hst[1] > 0 ? (float)((double)hst[0] / (double)hst[1] * 1e3) : 0.f;
        out->mma_tf32_sm_mhz = hst[3] > 0 ? (float)((double)hst[2] / (double)hst[3] * 1e3) : 0.f;
        if (host[1] != 0) s = kb_fail(ctx, KB_ERR_TIMEOUT, "kb_probe_peaks: %d CTAs did not see their products retire", host[1]);
    } while (0);
    if (s == KB_ERR_CUDA) kb_fail(ctx, KB_ERR_CUDA, "kb_probe_peaks: %s", cudaGetErrorString(cudaGetLastError()));
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    return s;
}
