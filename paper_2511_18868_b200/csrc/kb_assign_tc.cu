// kb_cluster_assign, tensor-core path (sm_100a: tcgen05.mma, TMEM).
//
// The assignment argmin_j ||z - c_j||^2 is a dense contraction Z[N x D] . C^T[D x K] when
// N*K*D is large.  It runs on the 5th-generation tensor cores as a three-product split
// (hi.hi + hi.lo + lo.hi, each operand split into two pieces of 11 significant bits by
// round-to-nearest, 22 bits in all), fp32 accumulate.  Two splits are built:
//
//   fp16 (default, kind::f16, 16 features per instruction).  fp16 and tf32 carry the same 11
//     significant bits, so the split is as exact as the tf32 one at half the tensor time.  fp16's
//     narrow exponent is handled by exact power-of-two scales: one per row (s_z), one per
//     instance for its centroids (s_c).  The constant terms ride along as 16 extra features
//     (pieces of s_z s_c ||z||^2 against 1, s_z / s_c against pieces of s_c^2 ||c||^2), so an
//     accumulator entry is g_i d2(i, j) with g_i = s_z s_c > 0 and the epilogue ranks the
//     accumulator as it is: no per-column constants, no floating-point work per column.
//   tf32 (kind::tf32, 8 features per instruction; kb_set_assign_options path 3).  No scales; the
//     epilogue forms ||z||^2 + ||c||^2 - 2 acc per column from the norms kept in shared memory.
//
//   * A = a 128-row tile of Z.  Every producer thread owns one row: it requests the row with one
//     bulk copy into its slot of the staging buffer, splits it hi/lo in registers and stores it
//     in TENSOR MEMORY (tcgen05.st); the MMA reads A from there (no shared-memory traffic for A,
//     and the three products of a k-step reuse it).
//   * B = 128 centroids x one 128-byte swizzle row of features per stage, pre-split hi/lo by a
//     small kernel into 128-byte-swizzled K-major panels, so a stage is one linear 32 KB bulk
//     copy (cp.async.bulk + mbarrier; the fp16 stage of a tile's first k-block also brings the
//     tile's 4 KB constant-term operand, K-major without swizzle), 4-stage ring, re-read from L2
//     by every CTA (no multicast of any kind).  The whole image stays resident when it fits.
//   * accumulators: two 128 x 128 fp32 buffers in TMEM; the epilogue warps read one with
//     tcgen05.ld while the MMA fills the other.
//   * epilogue: every value becomes an integer key that carries its column (tf32 split: the fp32 bits
//     with the low 7 bits replaced; fp16 split: a 22-bit fixed-point distance times KQ_MUL plus the
//     column), so integer min/max rank value and index together; per row the three smallest keys
//     are kept across all centroid tiles.  A row whose runner-up lies inside the error bound of
//     the split product is queued and decided in the exact direct form by a fix-up kernel (two
//     candidates: a warp compares them; three or more: all K are re-evaluated), so labels follow
//     the fp32 direct-form distances wherever it matters.
//
//   * pre-split image (template parameter APRE; inside kb_cluster_fit, fp16 split, D <= 64).  A fit assigns
//     the same Z many times, so it converts Z to its fp16 pieces ONCE (tc_prep_z_f16_kernel: per 128-row
//     tile a contiguous image of swizzled rows plus ||z||^2 and s_z per row) and its assignments run this
//     kernel with APRE: a fifth role brings a whole tile with one bulk copy (evict-first in L2) into a ring
//     of three, the producers only move their row from shared to tensor memory and form its constant-term
//     operand, and -- two tiles later -- take the row's candidates over from the epilogue through shared
//     memory, merge them, write the label and queue near-ties, so the epilogue goes straight on.
//
// Roles in a 448-thread persistent CTA (480 with APRE; one CTA per SM):
//   warps 0-3   A producers  (bulk copy of the next Z tile -> split -> TMEM; APRE: row image -> TMEM,
//                             constant terms, the rows' results two tiles behind)
//   warps 4-11  epilogue     (TMEM -> registers -> keys -> argmin; two warps per lane quarter)
//   warp  12    MMA issuer   (one elected lane), owns the TMEM allocation
//   warp  13    B loader     (one elected lane)
//   warp  14    A loader     (APRE only; one elected lane)
// The roles meet only at mbarriers (one arrival per warp).  Every wait is bounded and suspends
// the waiting thread between polls; on expiry the CTA raises an abort flag, all roles drain,
// copies in flight are awaited, TMEM is released and the device status word reports a timeout.
#include "kb_internal.cuh"
#include <cuda_fp16.h>

namespace {

constexpr int BM = 128;            // rows per tile = TMEM lanes
constexpr int BN = 128;            // centroids per accumulator buffer
constexpr int KBF = 32;            // floats per k-block (one 128-byte swizzle row)
constexpr int PANEL = BN * KBF * 4;      // 16 KB: one hi or lo panel
constexpr int STAGE = 2 * PANEL;         // hi + lo
constexpr int EXT = 4096;                // fp16 split: the constant-term operand of one centroid tile (128 x 16 halfs)
constexpr int SLOT_F16 = STAGE + EXT;    // a stage slot of the fp16 kernel (a multiple of 1024 bytes)
constexpr int XCOLS = 8;                 // TMEM columns of a row's constant-term operand (16 halfs)
constexpr int PREP_MAXG = 64;             // blocks per instance of the fp16 preparation kernel (at most)
constexpr int INST_STRIDE = 1 + PREP_MAXG; // floats per instance: s_c, then every preparation block's largest ||c||^2
constexpr int NSTAGE = 4;
constexpr int TC_THREADS = 448;
constexpr int TC_THREADS_APRE = 480;     // pre-split A: one more warp, which loads the A panels
constexpr int AINFO = BM * 8;             // bytes of a tile's row table (||z||^2, s_z per row)
constexpr int TMEM_COLS = 512;
constexpr int COL_ACC = 0;         // two accumulators: columns [0,128) and [128,256)
constexpr int COL_A = 256;         // A buffers from here: hi part | lo part (| constant terms), two buffers when they fit
constexpr uint32_t WAIT_LIMIT = 1u << 19;          // polls of a bounded wait, each suspended for up to WAIT_SUSPEND_NS
constexpr uint32_t WAIT_SUSPEND_NS = 2000;
constexpr int STATUS_TIMEOUT = 0x100;

// ---- PTX helpers ------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// One arrival for the whole warp: every lane's earlier work (shared-memory stores, completed
// tensor-memory loads/stores followed by the tcgen05 fence) is ordered before it by the warp
// barrier.  Barriers signalled this way count warps, not threads: 32 times fewer shared-memory
// atomics on the path between the roles.
__device__ __forceinline__ void mbar_arrive_warp(uint32_t bar) {
    __syncwarp();
    if ((threadIdx.x & 31) == 0) mbar_arrive(bar);
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// mbarrier.try_wait may keep the thread suspended for a system-dependent time while the phase is incomplete;
// where a role only wants to know whether it could go on, and has other work if it cannot, it asks with
// test_wait, which answers at once.
__device__ __forceinline__ bool mbar_test(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// The same test, but the hardware may keep the thread suspended for up to `ns` nanoseconds while
// the phase is incomplete (it resumes at once when the phase completes).  A waiting role then
// executes one instruction per `ns` instead of spinning, which matters here: the waiting roles
// share their schedulers with the epilogue warps.
__device__ __forceinline__ bool mbar_try_suspend(uint32_t bar, uint32_t parity, uint32_t ns) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity), "r"(ns)
        : "memory");
    return ok != 0;
}
// Bounded wait (about a second at most).  Returns false (and raises the CTA's abort flag) when
// the limit is hit or another role has already aborted.
// (abort_flag[1] holds the limit in polls: WAIT_LIMIT unless a test shortened it.)
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
    if (mbar_try(bar, parity)) return true;
    const uint32_t limit = (uint32_t)abort_flag[1];
    for (uint32_t i = 0; i < limit; ++i) {
        if (mbar_try_suspend(bar, parity, WAIT_SUSPEND_NS)) return true;
        if ((i & 7u) == 7u && *abort_flag) return false;
    }
    *abort_flag = 1;
    return false;
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}

// The same copy for data that is read once per kernel and is large (the pre-split image of Z): its lines
// are marked evict-first in L2, so that streaming them does not push out what later kernels re-read.
__device__ __forceinline__ void bulk_g2s_stream(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    uint64_t policy;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar), "l"(policy)
                 : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem desc], kind::tf32
template <bool F16>
__device__ __forceinline__ void tc_mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                          uint32_t accumulate) {
    if (F16)
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "setp.ne.b32 p, %4, 0;\n\t"
            "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
            ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
            : "memory");
    else
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "setp.ne.b32 p, %4, 0;\n\t"
            "tcgen05.mma.cta_group::1.kind::tf32 [%0], [%1], %2, %3, p;\n\t}"
            ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
            : "memory");
}
// accumulate form (enable_input_d is the constant true predicate)
template <bool F16>
__device__ __forceinline__ void tc_mma_ts_acc(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc) {
    if (F16)
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "setp.eq.b32 p, 0, 0;\n\t"
            "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
            ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc)
            : "memory");
    else
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "setp.eq.b32 p, 0, 0;\n\t"
            "tcgen05.mma.cta_group::1.kind::tf32 [%0], [%1], %2, %3, p;\n\t}"
            ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc)
            : "memory");
}
// true in exactly one lane of a converged warp
__device__ __forceinline__ bool elect_one() {
    uint32_t pred;
    asm volatile("{\n\t.reg .pred P;\n\telect.sync _|P, 0xffffffff;\n\tselp.u32 %0, 1, 0, P;\n\t}" : "=r"(pred));
    return pred != 0;
}
__device__ __forceinline__ uint64_t mk_desc(uint32_t lo, uint32_t hi) {
    return ((uint64_t)hi << 32) | (uint64_t)lo;
}
__device__ __forceinline__ uint32_t to_tf32(float v) {
    uint32_t r;
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(r) : "f"(v));
    return r;
}

#define TC_LD32(taddr, r)                                                                                  \
    asm volatile(                                                                                          \
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "                                                          \
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "                          \
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"          \
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),  \
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]),         \
          "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]),       \
          "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]),       \
          "=r"(r[29]), "=r"(r[30]), "=r"(r[31])                                                            \
        : "r"(taddr)                                                                                       \
        : "memory")

// The loaded registers are only valid after tcgen05.wait::ld; naming them as read-write
// operands of the wait keeps the compiler from consuming them earlier.
#define TC_WAIT_LD(r)                                                                                      \
    asm volatile("tcgen05.wait::ld.sync.aligned;"                                                          \
        : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]),  \
          "+r"(r[8]), "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]),         \
          "+r"(r[15]), "+r"(r[16]), "+r"(r[17]), "+r"(r[18]), "+r"(r[19]), "+r"(r[20]), "+r"(r[21]),       \
          "+r"(r[22]), "+r"(r[23]), "+r"(r[24]), "+r"(r[25]), "+r"(r[26]), "+r"(r[27]), "+r"(r[28]),       \
          "+r"(r[29]), "+r"(r[30]), "+r"(r[31])                                                            \
        :: "memory")

#define TC_ST32(taddr, r)                                                                                  \
    asm volatile(                                                                                          \
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "                                                    \
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "                         \
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"                 \
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]),         \
          "r"(r[7]), "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]),     \
          "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]),  \
          "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]),  \
          "r"(r[31])                                                                                       \
        : "memory")

// K-major, 128-byte swizzle: rows of 128 bytes, 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr) {
    uint64_t d = (uint64_t)((addr & 0x3FFFFu) >> 4);
    d |= (uint64_t)1 << 16;                 // leading byte offset (unused for swizzled K-major)
    d |= (uint64_t)(1024 >> 4) << 32;       // stride byte offset between 8-row groups
    d |= (uint64_t)1 << 46;                 // descriptor version for sm_100
    d |= (uint64_t)2 << 61;                 // SWIZZLE_128B
    return d;
}
// kind::tf32, fp32 accumulate, A and B K-major, M = 128, N = BN
constexpr uint32_t IDESC_TF32 = (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
// kind::f16 with fp16 operands (format 0), fp32 accumulate, same shape; one instruction covers K = 16
constexpr uint32_t IDESC_F16 = (1u << 4) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);


struct TcParams {
    int B, N, D, K, Kpad;
    int nkb;                       // k-blocks (128-byte swizzle rows) per centroid: D/32 tf32, ceil(D/64) fp16
    int DC;                        // TMEM columns of one A part (hi or lo): D for tf32, 32 * nkb for fp16
    int tiles_per_inst, total_tiles;
    int nxb;                       // Z staging buffers (1 or 2)
    int resident;                  // 1: the whole B image of the (single) instance stays in the stage ring
    float eps;                     // near-tie bound, relative to ||z||^2 + ||c||^2
    const float* z;
    const unsigned char* aimg;     // pre-split A: [tile][BM][row image], see tc_prep_z_f16_kernel
    const float* ainfo;            // pre-split A: [tile][BM][2]  ||z||^2 and s_z of every row
    int nstage_alloc;              // stage slots that exist in shared memory (the whole ring unless B is resident)
    const unsigned char* bimg;     // [B][NT][NKB][STAGE]
    const float* cnorm;            // [B][Kpad]
    const unsigned char* bext;     // fp16 split: [B][NT][EXT] constant-term operand of every centroid tile
    const float* inst;             // fp16 split: [B][INST_STRIDE] centroid scale s_c, then per-block largest ||c||^2
    int gprep;                     // blocks per instance the preparation kernel ran with
    int32_t* labels;
    float* approx;                 // optional: ||z||^2 + best score (expanded-form d^2), diagnostics
    int* flag_count;               // [0]: rows queued for a two-candidate check, [1]: for a full re-evaluation
    int2* pair_rows;               // (flat row id b * N + k, runner-up centroid)
    int32_t* full_rows;            // flat row ids
    int* dev_status;
    uint32_t wait_limit;           // polls of a bounded wait (WAIT_LIMIT; a test may shorten it)
    int absent_b_loader;           // test only: the B loader of CTA 0 never loads, so that CTA's waits run out
};

// ---- preparation: split centroids into swizzled hi/lo panels, squared norms ----------
// Power-of-two factor that brings a vector with largest magnitude m into [0.5, 1): the fp16 split
// keeps 22 significant bits only while hi and lo stay inside fp16's normal range, so every row
// and every centroid is scaled by its own exact factor and the product is unscaled afterwards.
__device__ __forceinline__ float pow2_scale(float m) {
    if (!(m > 0.f) || !(m < INFINITY)) return 1.f;
    // m = f 2^e with f in [0.5, 1): e is the biased exponent field minus 126 (a subnormal m has e < -126)
    const int field = (int)((__float_as_uint(m) >> 23) & 0xffu);
    int e = field == 0 ? -127 : field - 126;
    e = e < -100 ? -100 : (e > 100 ? 100 : e);
    return __uint_as_float((uint32_t)(127 - e) << 23);     // 2^-e
}
// (hi, lo) fp16 split of two scaled values, packed the way the tensor core reads 16-bit
// operands: the lower k index in the low half of the 32-bit word
__device__ __forceinline__ void split_f16x2(float a, float b, uint32_t& hi, uint32_t& lo) {
    const __half2 h = __floats2half2_rn(a, b);
    const float2 hf = __half22float2(h);
    const __half2 l = __floats2half2_rn(a - hf.x, b - hf.y);
    hi = *reinterpret_cast<const uint32_t*>(&h);
    lo = *reinterpret_cast<const uint32_t*>(&l);
}

// tf32 split: one warp per centroid, lane q owns the 16-byte chunk q of the fp32 row (D <= 128);
// hi/lo panels with 32 features per 128-byte swizzle row, squared norms in double.
__global__ void __launch_bounds__(256)
tc_prep_kernel(int K, int D, int Kpad, int nkb, const float* __restrict__ cent, unsigned char* __restrict__ bimg,
               float* __restrict__ cnorm, int* __restrict__ flag_count) {
    kb_grid_dependency_wait();
    if (blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x < 2) flag_count[threadIdx.x] = 0;   // empty both queues
    const int b = blockIdx.y;
    const int nt = Kpad / BN;
    const int lane = threadIdx.x & 31;
    const int j = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (j >= Kpad) return;
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    if (j < K && lane < D / 4) v = __ldg(reinterpret_cast<const float4*>(cent + ((size_t)b * K + j) * D) + lane);
    const float f[4] = {v.x, v.y, v.z, v.w};
    double sq = 0.0;
#pragma unroll
    for (int i = 0; i < 4; ++i) sq += (double)f[i] * (double)f[i];
    sq = kb_warp_sum(sq);
    if (lane < nkb * 8) {
        const int kb = lane >> 3, c = lane & 7;
        const int tile = j / BN, r = j - tile * BN;
        const size_t off = (((size_t)b * nt + tile) * nkb + kb) * STAGE + (size_t)(r >> 3) * 1024 + (r & 7) * 128 +
                           ((c ^ (r & 7)) << 4);
        uint32_t hi[4], lo[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            hi[i] = to_tf32(f[i]);
            lo[i] = to_tf32(f[i] - __uint_as_float(hi[i]));
        }
        *reinterpret_cast<uint4*>(bimg + off) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
        *reinterpret_cast<uint4*>(bimg + off + PANEL) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
    }
    if (lane == 0) cnorm[(size_t)b * Kpad + j] = j < K ? (float)sq : INFINITY;   // padding can never win
}

// Three fp16 pieces of a non-negative fp32 value (33 significant bits; a piece that falls below
// fp16's range simply contributes less, an absolute error far below the ranking bound).
__device__ __forceinline__ void split3_f16(float v, __half& a, __half& b, __half& c) {
    a = __float2half_rn(v);
    const float r1 = v - __half2float(a);
    b = __float2half_rn(r1);
    c = __float2half_rn(r1 - __half2float(b));
}
__device__ __forceinline__ uint32_t pack_h2(__half lo, __half hi) {
    return (uint32_t)__half_as_ushort(lo) | ((uint32_t)__half_as_ushort(hi) << 16);
}

// Preparation for the fp16 split with the constant terms folded into the product.
// With one power-of-two scale s_c per instance (largest |coordinate| of its centroids into
// [0.5, 1)) and one scale s_z per row, the tensor core is given
//     A row  i : s_z z_i (hi, lo)           | pieces of s_z s_c ||z_i||^2 | s_z / s_c (three times)
//     B row  j : -2 s_c c_j (hi, lo)        | 1, 1, 1                     | pieces of s_c^2 ||c_j||^2
// so that one accumulator entry is  s_z s_c (||z_i||^2 + ||c_j||^2 - 2 z_i.c_j)  =  g_i d2(i, j)  with
// g_i > 0: the epilogue ranks the accumulator as it is.  This kernel writes the B side:
//   bimg  [B][NT][nkb][hi panel | lo panel]   128-byte-swizzled K-major panels, 64 features per row
//   bext  [B][NT][EXT]   the 16 extra features of each centroid, K-major without swizzle
//                        (8-row x 16-byte core matrices: k-halves 128 bytes apart, row groups 256)
//   inst  [B][1 + blocks] s_c, then each block's largest ||c_j||^2 (plain stores: nothing to clear)
// Every block first scans its instance's centroids for the two maxima (the table is small and
// sits in L2), then converts its share of the centroids: one warp per centroid, lane q owns the
// 16-byte chunk q of the fp32 row (D <= 128).
__global__ void __launch_bounds__(256)
tc_prep_f16_kernel(int K, int D, int Kpad, int nkb, const float* __restrict__ cent, unsigned char* __restrict__ bimg,
                   unsigned char* __restrict__ bext, float* __restrict__ inst, int* __restrict__ flag_count) {
    kb_grid_dependency_wait();
    __shared__ float s_m[8];
    if (blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x < 2) flag_count[threadIdx.x] = 0;   // empty both queues
    const int b = blockIdx.y, nt = Kpad / BN;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const float* cb = cent + (size_t)b * K * D;
    // largest |coordinate| of the instance's centroids: every block scans the whole table (coalesced,
    // all loads independent), so that all of them derive the same scale without a grid-wide step
    float m = 0.f;
    {
        const float4* c4 = reinterpret_cast<const float4*>(cb);
        const int n4 = K * D / 4;
        for (int e = threadIdx.x; e < n4; e += 256) {
            const float4 v = __ldg(c4 + e);
            m = fmaxf(fmaxf(m, fmaxf(fabsf(v.x), fabsf(v.y))), fmaxf(fabsf(v.z), fabsf(v.w)));
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    if (lane == 0) s_m[warp] = m;
    __syncthreads();
#pragma unroll
    for (int w = 0; w < 8; ++w) m = fmaxf(m, s_m[w]);
    const float sc = pow2_scale(m);
    __shared__ float s_n[8];
    if (blockIdx.x == 0 && threadIdx.x == 0) inst[(size_t)b * INST_STRIDE] = sc;
    float nmax = 0.f;                                      // largest ||c_j||^2 among this warp's centroids

    for (int j = blockIdx.x * 8 + warp; j < Kpad; j += gridDim.x * 8) {
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (j < K && lane < D / 4) v = __ldg(reinterpret_cast<const float4*>(cb + (size_t)j * D) + lane);
        const double sq = kb_warp_sum((double)v.x * v.x + (double)v.y * v.y + (double)v.z * v.z + (double)v.w * v.w);
        nmax = fmaxf(nmax, (float)sq * 1.0000005f);
        const int tile = j / BN, r = j - tile * BN;
        if (lane < nkb * 16) {
            const int kb = lane >> 4, within = (lane & 15) * 8;            // byte offset inside the 128-byte row
            const size_t off = (((size_t)b * nt + tile) * nkb + kb) * STAGE + (size_t)(r >> 3) * 1024 + (r & 7) * 128 +
                               (((within >> 4) ^ (r & 7)) << 4) + (within & 15);
            const float w = -2.f * sc;
            uint32_t h0, l0, h1, l1;
            split_f16x2(v.x * w, v.y * w, h0, l0);
            split_f16x2(v.z * w, v.w * w, h1, l1);
            *reinterpret_cast<uint2*>(bimg + off) = make_uint2(h0, h1);
            *reinterpret_cast<uint2*>(bimg + off + PANEL) = make_uint2(l0, l1);
        }
        if (lane == 0) {
            const __half one = __float2half_rn(1.f), zero = __float2half_rn(0.f);
            __half q0 = __float2half_rn(INFINITY), q1 = zero, q2 = zero;   // a padding centroid can never win
            if (j < K) split3_f16((float)((double)sc * (double)sc * sq), q0, q1, q2);
            unsigned char* e = bext + ((size_t)b * nt + tile) * EXT + (size_t)(r >> 3) * 256 + (r & 7) * 16;
            *reinterpret_cast<uint4*>(e) = make_uint4(pack_h2(one, one), pack_h2(one, q0), pack_h2(q1, q2), 0u);
            *reinterpret_cast<uint4*>(e + 128) = make_uint4(0u, 0u, 0u, 0u);
        }
    }
    // this block's largest squared norm; the contraction kernel takes the maximum over the blocks
    if (lane == 0) s_n[warp] = nmax;
    __syncthreads();
    if (threadIdx.x == 0) {
#pragma unroll
        for (int w = 0; w < 8; ++w) nmax = fmaxf(nmax, s_n[w]);
        inst[(size_t)b * INST_STRIDE + 1 + blockIdx.x] = nmax;
    }
}

// The A side of the fp16 split, made ONCE for a matrix Z that many assignments will read (the Lloyd
// loop of a fit).  Every 128-row tile becomes one contiguous image,
//   aimg  [tile][128 rows][per k-block: 64 hi halfs | 64 lo halfs]
//         the fp16 pieces of s_z z (s_z brings the row's largest magnitude into [0.5, 1)), each row
//         in the order the tensor core reads a 16-bit A operand from tensor memory, except that the
//         eight 16-byte chunks of a piece are stored at chunk index ^ (row & 7)
//   ainfo [tile][128][2]   ||z||^2 and s_z of every row
// so that an assignment fetches a tile with ONE bulk copy and its row threads only move their row
// from shared to tensor memory (the chunk swizzle keeps their 16-byte reads free of bank conflicts); the
// row's constant-term operand, which depends on the centroids' scale, is still formed per assignment.
// Rows past the end of an instance are zeros.
__host__ __device__ constexpr int a_row_bytes(int nkb) { return nkb * 256; }

__global__ void __launch_bounds__(256)
tc_prep_z_f16_kernel(int N, int D, int nkb, int tiles_per_inst, const float* __restrict__ z,
                     unsigned char* __restrict__ aimg, float* __restrict__ ainfo) {
    kb_grid_dependency_wait();
    // a group of LPR lanes owns a row (lane q of the group: the 16-byte chunk q of the fp32 row, or zeros
    // behind the row's end up to the k-block's 64 features), RPW rows per warp
    const int LPR = nkb * 16, RPW = 32 / LPR;
    const int b = blockIdx.y, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int q = lane % LPR;
    const long slot = ((long)blockIdx.x * 8 + warp) * RPW + lane / LPR;    // row slot inside the instance's tiles
    const bool live = slot < (long)tiles_per_inst * BM;
    const int t = (int)(slot / BM), r = (int)(slot - (long)t * BM);
    const size_t tile = (size_t)b * tiles_per_inst + t;
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    if (live && slot < N && q < D / 4) v = __ldg(reinterpret_cast<const float4*>(z + ((size_t)b * N + slot) * D) + q);
    float xn = fmaf(v.w, v.w, fmaf(v.z, v.z, fmaf(v.y, v.y, v.x * v.x)));
    float m = fmaxf(fmaxf(fabsf(v.x), fabsf(v.y)), fmaxf(fabsf(v.z), fabsf(v.w)));
    for (int o = LPR >> 1; o > 0; o >>= 1) {
        xn += __shfl_xor_sync(0xffffffffu, xn, o);
        m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    }
    if (!live) return;
    const float sz = pow2_scale(m);
    unsigned char* row = aimg + (tile * BM + r) * (size_t)a_row_bytes(nkb);
    {
        const int kb = q >> 4, within = (q & 15) * 8;                      // byte offset inside the 128 bytes of a piece
        const int pos = (((within >> 4) ^ (r & 7)) << 4) + (within & 15);  // the same, with the chunk swizzled
        uint32_t h0, l0, h1, l1;
        split_f16x2(v.x * sz, v.y * sz, h0, l0);
        split_f16x2(v.z * sz, v.w * sz, h1, l1);
        *reinterpret_cast<uint2*>(row + kb * 256 + pos) = make_uint2(h0, h1);
        *reinterpret_cast<uint2*>(row + kb * 256 + 128 + pos) = make_uint2(l0, l1);
    }
    if (q == 0) *reinterpret_cast<float2*>(ainfo + (tile * BM + r) * 2) = make_float2(xn, sz);
}

// ---- the contraction -------------------------------------------------------------------
// Running smallest squared distances of one row, kept as integer KEYS: the fp32 bits of
// d2 = ||z||^2 + ||c||^2 - 2 z.c with the low KEY_BITS replaced by the column's index inside
// the 128-column accumulator tile.  Positive floats order like their bit patterns, so one
// integer min/max both ranks the value and carries the index along (no compare+select per
// column); dropping KEY_BITS mantissa bits moves a value by less than 2^-16 of itself, which the
// near-tie bound absorbs.  A d2 that rounding made slightly negative is a negative integer: it
// beats every positive key, and any two such values are closer than the near-tie bound, so the
// exact fix-up decides between them.
// TRACK2 keeps the three smallest keys (a near-tie between exactly two candidates is settled by
// comparing those two); without it only the two smallest are kept and every near-tie is
// re-evaluated against all centroids (cheaper per column; used when K*D is small).
constexpr int KEY_BITS = 7;
constexpr int KEY_MASK = ~((1 << KEY_BITS) - 1);
constexpr int KEY_INF = 0x7fffffff;
// fp16 split: the accumulator g_i d2 is turned into a FIXED-POINT key instead.  One FFMA maps it onto
// [2^23, 2^23 + 2^22) (the row's largest possible value, 2 g_i (||z||^2 + max ||c||^2), lands on the
// top), whose fp32 bits are 0x4B000000 + n with n the 22-bit quantised distance; one integer
// multiply-add turns the bits into n * KQ_MUL + column.  Both run on the FMA pipe, which the
// epilogue leaves idle, while the integer/logic pipe is what bounds the kernel.  KQ_MUL is odd and
// above 64 so that the product is not rewritten as shifts.
constexpr uint32_t KQ_MUL = 157u;
constexpr float KQ_TOP = 4194303.f;                                  // 2^22 - 1
constexpr uint32_t KQ_BASE = 0u - 0x4B000000u * KQ_MUL;              // removes the bits of 2^23
static_assert(BN == (1 << KEY_BITS), "a key's index field addresses one accumulator tile");

template <bool TRACK2>
struct KeyTracker {
    int b0 = KEY_INF, b1 = KEY_INF, b2 = KEY_INF;
    // two more columns: five (eight with TRACK2) integer min/max operations per pair
    __device__ __forceinline__ void add2(int k, int k2) {
        const int lo = min(k, k2), hi = max(k, k2);
        if (TRACK2) b2 = __vimin3_s32(b2, max(b1, lo), max(b0, hi));
        b1 = __vimin3_s32(b1, max(b0, lo), hi);
        b0 = min(b0, lo);
    }
    // fold another tracker over a disjoint set of columns into this one
    __device__ __forceinline__ void merge(const KeyTracker& u) {
        if (TRACK2) b2 = min(__vimin3_s32(b2, u.b2, max(b1, u.b0)), max(b0, u.b1));
        b1 = __vimin3_s32(b1, u.b1, max(b0, u.b0));
        b0 = min(b0, u.b0);
    }
};

// The smallest keys of a row across accumulator tiles, each with the tile it came from.
template <bool TRACK2>
struct RowBest {
    int r0 = KEY_INF, r1 = KEY_INF, r2 = KEY_INF;
    int t0 = 0, t1 = 0;
    __device__ __forceinline__ void insert(int k, int tile) {
        const bool c0 = k < r0, c1 = k < r1;
        if (TRACK2) {
            r2 = c1 ? r1 : min(r2, k);
            t1 = c0 ? t0 : (c1 ? tile : t1);
        }
        r1 = c0 ? r0 : (c1 ? k : r1);
        t0 = c0 ? tile : t0;
        r0 = c0 ? k : r0;
    }
    __device__ __forceinline__ float value(int key) const { return __int_as_float(key & KEY_MASK); }
    __device__ __forceinline__ int column(int key, int tile) const { return tile * BN + (key & ~KEY_MASK); }
};

// fp16 split: what a row's three smallest keys decide.  key = n * KQ_MUL + column (column inside the
// thread's 64; the tile id carries the half); n * kstep is the squared distance.  A slightly negative
// distance gives a negative key: it ranks first and reads as zero.  Writes the label (and the
// diagnostic distance) and queues the row for the exact re-evaluation when its runner-up lies inside
// the error bound.
// FINE: each of a thread's two trackers (alternate column pairs, 32 columns of the tile) handed over its
// own two smallest keys; otherwise the thread's trackers were merged first (64 columns per sub-chunk).
template <bool FINE>
__device__ __forceinline__ void emit_row_f16(const TcParams& p, const RowBest<true>& rb, size_t flat, float xn,
                                             float cmaxn, float rscale) {
    const float range_d2 = fmaxf(2.f * (xn + cmaxn), 1e-30f);
    const float kstep = range_d2 * (1.f / KQ_TOP);
    auto quant = [](int key) {             // floor division: a negative key keeps its column
        return key >= 0 ? key / (int)KQ_MUL : -((-key + (int)KQ_MUL - 1) / (int)KQ_MUL);
    };
    const int n0 = quant(rb.r0), n1 = quant(rb.r1), n2 = quant(rb.r2);
    const int l0 = rb.r0 - n0 * (int)KQ_MUL, l1 = rb.r1 - n1 * (int)KQ_MUL;
    const int a0 = (rb.t0 >> 1) * BN + (rb.t0 & 1) * (BN / 2) + l0;
    const int a1 = (rb.t1 >> 1) * BN + (rb.t1 & 1) * (BN / 2) + l1;
    const float b0 = (float)max(n0, 0) * kstep, b1 = (float)max(n1, 0) * kstep, b2 = (float)max(n2, 0) * kstep;
    // near-tie bound: the split product's error, relative to ||z||^2 plus the largest centroid norm of
    // the instance (its centroids share one scale), plus two quantisation steps
    const float delta = p.eps * (xn + cmaxn) + 2.f * kstep;
    // the third smallest is only known when the two smallest come from different sub-chunks (each
    // sub-chunk hands over its two smallest keys only)
    const bool third_known = FINE ? !(rb.t0 == rb.t1 && ((l0 ^ l1) & 2) == 0) : rb.t0 != rb.t1;
    p.labels[flat] = a0;
    if (p.approx) p.approx[flat] = b0;
    if (rscale < 0.f) {                                // row outside the fp16 range: exact scan over all K
        const int slot = atomicAdd(p.flag_count + 1, 1);
        p.full_rows[slot] = (int32_t)flat;
    } else if (fabsf(b1 - b0) <= delta) {
        if (third_known && fabsf(b2 - b0) > delta) {   // exactly two candidates: compare them exactly
            const int slot = atomicAdd(p.flag_count, 1);
            p.pair_rows[slot] = make_int2((int)flat, a1);
        } else {                                       // three or more (or unknown): exact scan over all K
            const int slot = atomicAdd(p.flag_count + 1, 1);
            p.full_rows[slot] = (int32_t)flat;
        }
    }
}

template <bool TRACK2, bool F16, bool APRE>
__global__ void __launch_bounds__(APRE ? TC_THREADS_APRE : TC_THREADS, 1)
assign_tc_kernel(const TcParams p) {
    static_assert(!APRE || F16, "the pre-split A image exists for the fp16 split only");
    // fp16 split: the hot loop keeps the two smallest keys of each sub-chunk (the 32 columns one
    // tracker sees in an accumulator tile; the pre-split kernel merges a thread's two trackers: 64
    // columns); the row's running best keeps three keys.  The third
    // smallest distance of the row is then known unless the two smallest come from the same
    // sub-chunk, in which case a near-tie goes to the full re-evaluation.
    constexpr bool HOT3 = F16 ? false : TRACK2;           // hot-loop trackers keep a third key
    constexpr bool ROW3 = F16 ? true : TRACK2;            // the running best keeps three keys, two tiles
    extern __shared__ unsigned char smem_raw[];
    // 1024-byte alignment for the swizzled panels
    unsigned char* smem = reinterpret_cast<unsigned char*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const int D = p.D, nkb = p.nkb, nt_count = p.Kpad / BN;
    const int DC = p.DC;                                  // TMEM columns of one A part (hi or lo)
    const int AST = 2 * DC + (F16 ? XCOLS : 0);           // TMEM columns of one A buffer: hi | lo | constant terms
    const int nab = 2 * AST <= 256 ? 2 : 1;               // A buffers that fit beside the accumulators in TMEM
    constexpr int SLOT = F16 ? SLOT_F16 : STAGE;          // bytes of one stage slot
    const int xs_stride = D + 4;                          // floats; keeps float4 row reads conflict-free
    unsigned char* st_base = smem;                                        // nstage_alloc x SLOT
    float* xs = reinterpret_cast<float*>(smem + (size_t)p.nstage_alloc * SLOT);   // nxb x [BM][D+4]
    // pre-split A: nxb x [BM][row image], then nxb x [BM][2] row tables, instead of xs
    unsigned char* as_base = smem + (size_t)p.nstage_alloc * SLOT;
    const int ARB = a_row_bytes(nkb), ABUF = BM * ARB;                    // bytes of a row image, of a tile's
    float* as_info = reinterpret_cast<float*>(as_base + (size_t)p.nxb * ABUF);
    float* cn = APRE ? as_info + (size_t)p.nxb * BM * 2                   // tf32: [B][Kpad] norms; fp16: [B][2] (s_c, max norm)
                     : xs + (size_t)p.nxb * BM * xs_stride;
    float* xnorm = cn + (F16 ? (size_t)2 * p.B : (size_t)p.B * p.Kpad);   // [2][BM]
    float* xscale = xnorm + 2 * BM;                                       // [2][BM]  fp16: the row's key factor (negative: row out of range)
    float* merge_buf = xscale + 2 * BM;                                   // [2][2][BM][5]  (tile parity, half, row)
    uint64_t* bars = reinterpret_cast<uint64_t*>(merge_buf + 4 * BM * 5 + 2);   // (+2 floats: 8-byte alignment)
    // barrier indices
    enum { B_FULL = 0, B_EMPTY = NSTAGE, A_FULL = 2 * NSTAGE, A_EMPTY = A_FULL + 8, ACC_FULL = A_EMPTY + 8,
           ACC_EMPTY = ACC_FULL + 2, XN_FULL = ACC_EMPTY + 2, XN_EMPTY = XN_FULL + 2, X_FULL = XN_EMPTY + 2,
           AS_EMPTY = X_FULL + 3, MG_FULL = AS_EMPTY + 3, MG_FREE = MG_FULL + 2, NBAR = MG_FREE + 2 };
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + NBAR);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t bar0 = smem_u32(bars);
    auto BAR = [&](int i) { return bar0 + 8u * (uint32_t)i; };

    if (tid == 0) {
        for (int s = 0; s < NSTAGE; ++s) { mbar_init(BAR(B_FULL + s), 1); mbar_init(BAR(B_EMPTY + s), 1); }
        for (int k = 0; k < 8; ++k) { mbar_init(BAR(A_FULL + k), 4); mbar_init(BAR(A_EMPTY + k), 1); }
        for (int k = 0; k < 2; ++k) {
            mbar_init(BAR(ACC_FULL + k), 1); mbar_init(BAR(ACC_EMPTY + k), 8);
            mbar_init(BAR(XN_FULL + k), 4); mbar_init(BAR(XN_EMPTY + k), 8);
        }
        // staged rows: one arrival per producer thread; pre-split A: the loader's expect-tx arrival
        for (int k = 0; k < 3; ++k) { mbar_init(BAR(X_FULL + k), APRE ? 1 : 128); mbar_init(BAR(AS_EMPTY + k), 4); }
        // pre-split A: the epilogue hands every row's candidates to the row's thread among warps 0-3
        for (int k = 0; k < 2; ++k) { mbar_init(BAR(MG_FULL + k), 8); mbar_init(BAR(MG_FREE + k), 4); }
        abort_flag[0] = 0;
        abort_flag[1] = (int)p.wait_limit;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 12) {  // TMEM allocation (whole warp), address lands in shared memory
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(tmem_slot)), "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    // everything above touches only this CTA's shared and tensor memory: it may overlap the tail of
    // the preceding kernel; from here on its results are read
    kb_grid_dependency_wait();
    if (F16) {
        for (int j = tid; j < p.B; j += (int)blockDim.x) {                     // per instance: s_c, largest ||c||^2
            const float* ib = p.inst + (size_t)j * INST_STRIDE;
            float nm = 0.f;
            for (int g = 0; g < p.gprep; ++g) nm = fmaxf(nm, ib[1 + g]);
            cn[2 * j] = ib[0];
            cn[2 * j + 1] = nm;
        }
    } else {
        for (int j = tid; j < p.B * p.Kpad; j += (int)blockDim.x) cn[j] = p.cnorm[j];   // all instances' centroid norms
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    const int first = blockIdx.x, stride = gridDim.x;
    bool ok = true;

    if (APRE && warp < 4) {
        // ============================ A from the pre-split image ======================
        // The tile arrives pre-split by one bulk copy; each thread moves its row from shared to tensor
        // memory and forms the row's constant-term operand (it depends on the centroids' scale s_c) and
        // the two numbers the epilogue wants.
        const int row_in_tile = tid;                       // = TMEM lane
        const uint32_t lane_addr = tmem + ((uint32_t)(warp * 32) << 16);
        // What the epilogue found for this thread's row of tile number `jt` (of this CTA): merge the two
        // halves' candidates, write the label, queue a near-tie.
        auto finish_row = [&](int jt, int tile, float xn, float rscale) -> bool {
            if (!mbar_wait(BAR(MG_FULL + (jt & 1)), (uint32_t)((jt >> 1) & 1), abort_flag)) return false;
            const float* m0 = merge_buf + ((size_t)((jt & 1) * 2) * BM + row_in_tile) * 5;
            const float* m1 = m0 + BM * 5;
            RowBest<true> rb;
            rb.r0 = __float_as_int(m0[0]); rb.r1 = __float_as_int(m0[1]); rb.r2 = __float_as_int(m0[2]);
            rb.t0 = __float_as_int(m0[3]); rb.t1 = __float_as_int(m0[4]);
            const int u0 = __float_as_int(m1[0]), u1 = __float_as_int(m1[1]), u2 = __float_as_int(m1[2]);
            const int v0 = __float_as_int(m1[3]), v1 = __float_as_int(m1[4]);
            mbar_arrive_warp(BAR(MG_FREE + (jt & 1)));
            rb.insert(u0, v0);
            rb.insert(u1, v1);
            rb.r2 = min(rb.r2, u2);
            const int b = tile / p.tiles_per_inst, row = (tile - b * p.tiles_per_inst) * BM + row_in_tile;
            if (row < p.N) emit_row_f16<false>(p, rb, (size_t)b * p.N + row, xn, cn[2 * b + 1], rscale);
            return true;
        };
        // rows are finished two tiles behind: the constant terms of tile i + 1 must be in place when the
        // epilogue hands back the first accumulator of tile i, long before it is through with tile i - 1
        int it = 0, tile1 = -1, tile2 = -1;                // the previous tile and the one before it
        float xn1 = 0.f, rs1 = 1.f, xn2 = 0.f, rs2 = 1.f;
        for (int tile = first; tile < p.total_tiles && ok; tile += stride, ++it) {
            const int buf = it % p.nxb, ab = it % nab, use = it / nab;
            ok = mbar_wait(BAR(X_FULL + buf), (uint32_t)((it / p.nxb) & 1), abort_flag);
            if (!ok) break;
            const float2 info = *reinterpret_cast<const float2*>(as_info + ((size_t)buf * BM + row_in_tile) * 2);
            const float xn = info.x, sz = info.y;
            const float s_c = cn[2 * (tile / p.tiles_per_inst)];
            float rho = sz / s_c;                                  // both powers of two: exact
            const float g = sz * s_c;
            float pterm = g * xn;                                  // s_z s_c ||z||^2
            // a row far outside the centroids' range (s_z / s_c outside fp16's normal range, or a norm
            // term that would overflow fp16) is handed to the exact re-evaluation
            const bool out_of_range = !(rho >= 6.103515625e-05f && rho <= 16384.f) || !(pterm < 60000.f);
            const float rscale = out_of_range ? -1.f : 1.f / g;
            if (out_of_range) { rho = 0.f; pterm = 0.f; }
            const unsigned char* xr = as_base + (size_t)buf * ABUF + (size_t)row_in_tile * ARB;
            for (int kb = 0; kb < nkb && ok; ++kb) {
                uint32_t hi[32], lo[32];
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                    const int pos = (q ^ (row_in_tile & 7)) << 4;      // chunk q of the piece, where the image keeps it
                    const uint4 h = *reinterpret_cast<const uint4*>(xr + kb * 256 + pos);
                    const uint4 l = *reinterpret_cast<const uint4*>(xr + kb * 256 + 128 + pos);
                    hi[4 * q] = h.x; hi[4 * q + 1] = h.y; hi[4 * q + 2] = h.z; hi[4 * q + 3] = h.w;
                    lo[4 * q] = l.x; lo[4 * q + 1] = l.y; lo[4 * q + 2] = l.z; lo[4 * q + 3] = l.w;
                }
                ok = mbar_wait(BAR(A_EMPTY + ab * 4 + kb), (uint32_t)((use & 1) ^ 1), abort_flag);
                if (!ok) break;
                tc_fence_after();
                TC_ST32(lane_addr + COL_A + ab * AST + kb * 32, hi);
                TC_ST32(lane_addr + COL_A + ab * AST + DC + kb * 32, lo);
                if (kb == 0) {     // the row's constant-term operand travels with the first k-block
                    __half p0, p1, p2;
                    split3_f16(pterm, p0, p1, p2);
                    const __half hr = __float2half_rn(rho);
                    const uint32_t e0 = pack_h2(p0, p1), e1 = pack_h2(p2, hr), e2 = pack_h2(hr, hr), ez = 0u;
                    asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
                                 ::"r"(lane_addr + COL_A + ab * AST + 2 * DC), "r"(e0), "r"(e1), "r"(e2), "r"(ez), "r"(ez),
                                   "r"(ez), "r"(ez), "r"(ez)
                                 : "memory");
                }
                asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
                tc_fence_before();
                mbar_arrive_warp(BAR(A_FULL + ab * 4 + kb));
            }
            if (!ok) break;
            mbar_arrive_warp(BAR(AS_EMPTY + buf));                 // the row image has been read: the slot may be refilled
            ok = mbar_wait(BAR(XN_EMPTY + (it & 1)), (uint32_t)(((it >> 1) & 1) ^ 1), abort_flag);
            if (!ok) break;
            xnorm[(it & 1) * BM + row_in_tile] = xn;
            // the factor that maps an accumulator value onto the key range (the row's largest possible
            // value, 2 g (||z||^2 + max ||c||^2), lands on the top)
            xscale[(it & 1) * BM + row_in_tile] =
                KQ_TOP * fabsf(rscale) / fmaxf(2.f * (xn + cn[2 * (tile / p.tiles_per_inst) + 1]), 1e-30f);
            mbar_arrive_warp(BAR(XN_FULL + (it & 1)));
            if (tile2 >= 0) ok = finish_row(it - 2, tile2, xn2, rs2);
            tile2 = tile1; xn2 = xn1; rs2 = rs1;
            tile1 = tile; xn1 = xn; rs1 = rscale;
        }
        if (ok && tile2 >= 0) ok = finish_row(it - 2, tile2, xn2, rs2);
        if (ok && tile1 >= 0) ok = finish_row(it - 1, tile1, xn1, rs1);
    } else if (warp < 4) {
        // ============================ A producers ====================================
        const int row_in_tile = tid;                       // = TMEM lane
        const uint32_t lane_addr = tmem + ((uint32_t)(warp * 32) << 16);
        // Staging: every producer thread owns one row slot of the staging buffer.  It requests its
        // row with ONE bulk copy (the row is contiguous in global memory) that completes on the
        // buffer's mbarrier, and later reads only that slot, so a slot is never shared between
        // threads and needs no block-level barrier.  A row past the end of the instance is zeros.
        auto prefetch = [&](int tile, int buf) {
            const int b = tile / p.tiles_per_inst, r0 = (tile - b * p.tiles_per_inst) * BM;
            float* dst = xs + (size_t)buf * BM * xs_stride + (size_t)row_in_tile * xs_stride;
            if (r0 + row_in_tile < p.N) {
                mbar_expect_tx(BAR(X_FULL + buf), (uint32_t)D * 4u);
                bulk_g2s(smem_u32(dst), p.z + ((size_t)b * p.N + r0 + row_in_tile) * D, (uint32_t)D * 4u, BAR(X_FULL + buf));
            } else {
                for (int q = 0; q < D / 4; ++q) reinterpret_cast<float4*>(dst)[q] = make_float4(0.f, 0.f, 0.f, 0.f);
                mbar_arrive(BAR(X_FULL + buf));
            }
        };
        int it = 0;
        int uses0 = 0, uses1 = 0;                          // requests issued so far into staging buffer 0 / 1
        if (first < p.total_tiles) { prefetch(first, 0); ++uses0; }
        for (int tile = first; tile < p.total_tiles && ok; tile += stride, ++it) {
            const int buf = p.nxb == 2 ? (it & 1) : 0;
            const int next = tile + stride;
            if (p.nxb == 2 && next < p.total_tiles) {
                prefetch(next, buf ^ 1);
                if (buf) ++uses0; else ++uses1;
            }
            // this tile's rows have landed (request k into a buffer completes the barrier's phase k)
            ok = mbar_wait(BAR(X_FULL + buf), (uint32_t)((p.nxb == 2 ? (it >> 1) : it) & 1), abort_flag);
            if (!ok) break;
            const float* xr = xs + (size_t)buf * BM * xs_stride + (size_t)row_in_tile * xs_stride;
            float xn = 0.f, rscale = 1.f;
            const int ab = it % nab, use = it / nab;           // A buffer of this tile, how often it was used before
            if (F16) {
                // squared norm and largest magnitude of the row, then its power-of-two scale s_z: the
                // largest magnitude goes into [0.5, 1) unless that would put s_z / s_c outside fp16's
                // normal range
                float m = 0.f;
                for (int q = 0; q < D / 4; ++q) {
                    const float4 v = *reinterpret_cast<const float4*>(xr + 4 * q);
                    xn = fmaf(v.x, v.x, xn); xn = fmaf(v.y, v.y, xn); xn = fmaf(v.z, v.z, xn); xn = fmaf(v.w, v.w, xn);
                    m = fmaxf(fmaxf(m, fmaxf(fabsf(v.x), fabsf(v.y))), fmaxf(fabsf(v.z), fabsf(v.w)));
                }
                const int binst = tile / p.tiles_per_inst;
                const float s_c = cn[2 * binst];
                float rho = fminf(fmaxf(pow2_scale(m) / s_c, 6.103515625e-05f), 16384.f);   // s_z / s_c in [2^-14, 2^14]
                float sz = rho * s_c;
                const float g = sz * s_c;
                float pterm = g * xn;                              // s_z s_c ||z||^2
                // a row far outside the centroids' range (its scaled entries or its norm term would
                // overflow fp16) contributes zeros and is handed to the exact re-evaluation
                const bool out_of_range = !(m * sz < 32768.f) || !(pterm < 60000.f);
                rscale = out_of_range ? -1.f : 1.f / g;
                if (out_of_range) { sz = 0.f; rho = 0.f; pterm = 0.f; }
                for (int kb = 0; kb < nkb && ok; ++kb) {
                    uint32_t hi[32], lo[32];
                    const int nq = min(16, (D - kb * 64) / 4);     // float4 groups of this k-block that hold features
#pragma unroll
                    for (int q = 0; q < 16; ++q) {
                        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
                        if (q < nq) v = *reinterpret_cast<const float4*>(xr + kb * 64 + 4 * q);
                        split_f16x2(v.x * sz, v.y * sz, hi[2 * q], lo[2 * q]);
                        split_f16x2(v.z * sz, v.w * sz, hi[2 * q + 1], lo[2 * q + 1]);
                    }
                    ok = mbar_wait(BAR(A_EMPTY + ab * 4 + kb), (uint32_t)((use & 1) ^ 1), abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    TC_ST32(lane_addr + COL_A + ab * AST + kb * 32, hi);
                    TC_ST32(lane_addr + COL_A + ab * AST + DC + kb * 32, lo);
                    if (kb == 0) {     // the row's constant-term operand travels with the first k-block
                        __half p0, p1, p2;
                        split3_f16(pterm, p0, p1, p2);
                        const __half hr = __float2half_rn(rho);
                        const uint32_t e0 = pack_h2(p0, p1), e1 = pack_h2(p2, hr), e2 = pack_h2(hr, hr), ez = 0u;
                        asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
                                     ::"r"(lane_addr + COL_A + ab * AST + 2 * DC), "r"(e0), "r"(e1), "r"(e2), "r"(ez), "r"(ez),
                                       "r"(ez), "r"(ez), "r"(ez)
                                     : "memory");
                    }
                    asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
                    tc_fence_before();
                    mbar_arrive_warp(BAR(A_FULL + ab * 4 + kb));
                }
            } else {
            for (int kb = 0; kb < nkb && ok; ++kb) {
                uint32_t hi[32], lo[32];
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                    const float4 v = *reinterpret_cast<const float4*>(xr + kb * KBF + 4 * q);
                    const float f[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        xn = fmaf(f[i], f[i], xn);
                        hi[4 * q + i] = to_tf32(f[i]);
                        lo[4 * q + i] = to_tf32(f[i] - __uint_as_float(hi[4 * q + i]));
                    }
                }
                ok = mbar_wait(BAR(A_EMPTY + ab * 4 + kb), (uint32_t)((use & 1) ^ 1), abort_flag);
                if (!ok) break;
                tc_fence_after();
                TC_ST32(lane_addr + COL_A + ab * AST + kb * KBF, hi);
                TC_ST32(lane_addr + COL_A + ab * AST + DC + kb * KBF, lo);
                asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
                tc_fence_before();
                mbar_arrive_warp(BAR(A_FULL + ab * 4 + kb));
            }
            }
            if (!ok) break;
            if (p.nxb == 1 && next < p.total_tiles) { prefetch(next, 0); ++uses0; }   // own slot: already read
            ok = mbar_wait(BAR(XN_EMPTY + (it & 1)), (uint32_t)(((it >> 1) & 1) ^ 1), abort_flag);
            if (!ok) break;
            xnorm[(it & 1) * BM + row_in_tile] = xn;
            // fp16 split: the factor that maps an accumulator value onto the key range (the row's largest
            // possible value, 2 g (||z||^2 + max ||c||^2), lands on the top), negative for a row out of range
            if (F16) rscale = copysignf(KQ_TOP * fabsf(rscale) / fmaxf(2.f * (xn + cn[2 * (tile / p.tiles_per_inst) + 1]), 1e-30f), rscale);
            xscale[(it & 1) * BM + row_in_tile] = rscale;
            mbar_arrive_warp(BAR(XN_FULL + (it & 1)));
        }
        if (!ok) {
            // abort path: let row copies that may still be in flight land before shared memory goes
            // away (a phase that was already waited for answers at once)
            for (uint32_t i = 0; uses0 > 0 && i < WAIT_LIMIT && !mbar_try(BAR(X_FULL + 0), (uint32_t)((uses0 - 1) & 1)); ++i) {}
            for (uint32_t i = 0; uses1 > 0 && i < WAIT_LIMIT && !mbar_try(BAR(X_FULL + 1), (uint32_t)((uses1 - 1) & 1)); ++i) {}
        }
    } else if (warp < 12) {
        // ============================ epilogue ========================================
        // Two warps per TMEM lane quarter: `half` 0 takes columns [0,64) of every accumulator
        // buffer, `half` 1 columns [64,128).  Each thread keeps two independent key trackers per
        // accumulator tile (alternate column pairs) and folds them into the row's running best
        // after the accumulator buffer has been handed back to the MMA warp.
        const int ew = warp - 4, half = ew >> 2;
        const int row_in_tile = (ew & 3) * 32 + lane;
        const uint32_t lane_addr = tmem + ((uint32_t)((ew & 3) * 32) << 16);
        uint32_t q = 0;
        int it = 0;
        uint32_t r[2][32];                                   // two 32-column register buffers, reused in turn
        bool pref = false;                                   // the next tile's first load is already in flight
        for (int tile = first; tile < p.total_tiles && ok; tile += stride, ++it) {
            const int b = tile / p.tiles_per_inst, r0 = (tile - b * p.tiles_per_inst) * BM;
            const float* cnb = cn + (size_t)b * p.Kpad;            // squared norms of this instance's centroids
            // every epilogue thread takes the same waits in the same order, so a timeout takes
            // all of them out together and nobody is left at the named barrier below
            ok = mbar_wait(BAR(XN_FULL + (it & 1)), (uint32_t)((it >> 1) & 1), abort_flag);
            if (!ok) break;
            const float xn = xnorm[(it & 1) * BM + row_in_tile];
            const float rscale = xscale[(it & 1) * BM + row_in_tile];
            mbar_arrive_warp(BAR(XN_EMPTY + (it & 1)));
            RowBest<ROW3> rb;
            // fp16 split: quantisation step of the keys in units of d2, and the factor that maps an
            // accumulator value onto the key range
            const float cmaxn = F16 ? cn[2 * b + 1] : 0.f;
            const float kmul = fabsf(rscale);                      // fp16 split: the producer left the key factor here
            for (int nt = 0; nt < nt_count && ok; ++nt, ++q) {
                const uint32_t buf = q & 1u;
                const uint32_t acc = lane_addr + COL_ACC + buf * BN + half * (BN / 2);
                if (!pref) {                                   // first 32 columns not requested yet
                    ok = mbar_wait(BAR(ACC_FULL + buf), (q >> 1) & 1u, abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    TC_LD32(acc, r[0]);
                }
                pref = false;
                KeyTracker<HOT3> ta, tb;
                const float* cnp = cnb + nt * BN + half * (BN / 2);
                // Two passes over a 32-column register buffer.  The first turns every accumulator value
                // into its key in place: 32 independent short chains (load the column's constants,
                // three fp32 operations, one logic operation), which the scheduler can overlap freely.
                // The second feeds the keys to four independent trackers.
                auto process = [&](uint32_t (&v)[32], int c) {
#pragma unroll
                    for (int j = 0; j < 32; j += 4) {
                        const int l = c * 32 + j;                  // column inside this thread's 64
                        int k0, k1, k2, k3;
                        if (F16) {      // the accumulator already is g_i d2(i, j): quantise it and append the column
                            k0 = (int)(__float_as_uint(fmaf(__uint_as_float(v[j + 0]), kmul, 8388608.f)) * KQ_MUL + (KQ_BASE + (uint32_t)(l + 0)));
                            k1 = (int)(__float_as_uint(fmaf(__uint_as_float(v[j + 1]), kmul, 8388608.f)) * KQ_MUL + (KQ_BASE + (uint32_t)(l + 1)));
                            k2 = (int)(__float_as_uint(fmaf(__uint_as_float(v[j + 2]), kmul, 8388608.f)) * KQ_MUL + (KQ_BASE + (uint32_t)(l + 2)));
                            k3 = (int)(__float_as_uint(fmaf(__uint_as_float(v[j + 3]), kmul, 8388608.f)) * KQ_MUL + (KQ_BASE + (uint32_t)(l + 3)));
                        } else {
                            const float4 n4 = *reinterpret_cast<const float4*>(cnp + c * 32 + j);
                            k0 = (__float_as_int(fmaf(-2.f, __uint_as_float(v[j + 0]), n4.x + xn)) & KEY_MASK) | (l + 0);
                            k1 = (__float_as_int(fmaf(-2.f, __uint_as_float(v[j + 1]), n4.y + xn)) & KEY_MASK) | (l + 1);
                            k2 = (__float_as_int(fmaf(-2.f, __uint_as_float(v[j + 2]), n4.z + xn)) & KEY_MASK) | (l + 2);
                            k3 = (__float_as_int(fmaf(-2.f, __uint_as_float(v[j + 3]), n4.w + xn)) & KEY_MASK) | (l + 3);
                        }
                        ta.add2(k0, k1);
                        tb.add2(k2, k3);
                    }
                };
                TC_WAIT_LD(r[0]);
                TC_LD32(acc + 32, r[1]);
                process(r[0], 0);
                TC_WAIT_LD(r[1]);
                // both loads have landed: the accumulator goes back to the MMA warp before its second
                // half is even looked at
                tc_fence_before();
                mbar_arrive_warp(BAR(ACC_EMPTY + buf));
                // If the next accumulator tile is already complete (the usual case once the epilogue is
                // what the MMA warp waits for), request its first 32 columns now: the load then runs
                // under the arithmetic below instead of in front of the next tile's.
                const bool more = nt + 1 < nt_count || tile + stride < p.total_tiles;
                if (more) {
                    const uint32_t qn = q + 1u, bufn = qn & 1u;
                    if (__all_sync(0xffffffffu, mbar_test(BAR(ACC_FULL + bufn), (qn >> 1) & 1u))) {
                        tc_fence_after();
                        TC_LD32(lane_addr + COL_ACC + bufn * BN + half * (BN / 2), r[0]);
                        pref = true;
                    }
                }
                process(r[1], 1);
                if (F16) {
                    // the tile id carries the half
                    const int tid2 = nt * 2 + half;
                    if (APRE) {            // the two smallest keys of this thread's 64 columns: fewer inserts on the
                        ta.merge(tb);      // epilogue's chain, a few more rows in the full re-evaluation
                        rb.insert(ta.b0, tid2);
                        rb.insert(ta.b1, tid2);
                    } else {               // both trackers hand over their two smallest keys
                        rb.insert(ta.b0, tid2);
                        rb.insert(ta.b1, tid2);
                        rb.insert(tb.b0, tid2);
                        rb.insert(tb.b1, tid2);
                    }
                } else {
                    ta.merge(tb);
                    const int hbit = half * (BN / 2);              // the upper half's columns start at 64
                    rb.insert(ta.b0 | hbit, nt);
                    rb.insert(ta.b1 | hbit, nt);
                    if (TRACK2) rb.insert(ta.b2 | hbit, nt);
                }
            }
            if (!ok) break;
            if (APRE) {
                // both halves leave the row's candidates in shared memory for the row's thread among warps
                // 0-3, which has little else to do here, and go straight on to the next tile
                ok = mbar_wait(BAR(MG_FREE + (it & 1)), (uint32_t)(((it >> 1) & 1) ^ 1), abort_flag);
                if (!ok) break;
                float* mo = merge_buf + ((size_t)((it & 1) * 2 + half) * BM + row_in_tile) * 5;
                mo[0] = __int_as_float(rb.r0); mo[1] = __int_as_float(rb.r1); mo[2] = __int_as_float(rb.r2);
                mo[3] = __int_as_float(rb.t0); mo[4] = __int_as_float(rb.t1);
                mbar_arrive_warp(BAR(MG_FULL + (it & 1)));
                continue;
            }
            // fold the upper half's running best into the lower half's through shared memory
            float* mg = merge_buf + ((size_t)(it & 1) * BM + row_in_tile) * 5;
            if (half == 1) {
                mg[0] = __int_as_float(rb.r0); mg[1] = __int_as_float(rb.r1); mg[2] = __int_as_float(rb.r2);
                mg[3] = __int_as_float(rb.t0); mg[4] = __int_as_float(rb.t1);
            }
            asm volatile("bar.sync 2, 256;" ::: "memory");
            if (half == 1) continue;
            rb.insert(__float_as_int(mg[0]), __float_as_int(mg[3]));
            rb.insert(__float_as_int(mg[1]), __float_as_int(mg[4]));
            if (ROW3) rb.r2 = min(rb.r2, __float_as_int(mg[2]));
            const int row = r0 + row_in_tile;
            if (row < p.N) {
                const size_t flat = (size_t)b * p.N + row;
                if constexpr (F16) {
                    emit_row_f16<true>(p, rb, flat, xn, cmaxn, rscale);
                } else {
                    const int a0 = rb.column(rb.r0, rb.t0), a1 = rb.column(rb.r1, rb.t1);
                    const float b0 = rb.value(rb.r0), b1 = rb.value(rb.r1), b2 = rb.value(rb.r2);
                    // near-tie bound: the split product's error, relative to ||z||^2 plus the chosen
                    // centroid's norm, plus what the dropped key bits can hide
                    const float delta = p.eps * (xn + cnb[a0]) + 1.52587890625e-5f * fabsf(b1);
                    p.labels[flat] = a0;
                    if (p.approx) p.approx[flat] = b0;
                    if (fabsf(b1 - b0) <= delta) {
                        if (ROW3 && fabsf(b2 - b0) > delta) {      // exactly two candidates: compare them exactly
                            const int slot = atomicAdd(p.flag_count, 1);
                            p.pair_rows[slot] = make_int2((int)flat, a1);
                        } else {                                   // three or more (or unknown): exact scan over all K
                            const int slot = atomicAdd(p.flag_count + 1, 1);
                            p.full_rows[slot] = (int32_t)flat;
                        }
                    }
                }
            }
        }
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");   // no load may outlive the role (abort path)
    } else if (warp == 12) {
        // ============================ MMA issuer ======================================
        // One elected lane issues every MMA; the WHOLE warp runs the loop, and only the tcgen05
        // instructions sit under the elected-lane predicate (in warp-uniform control flow the
        // descriptor arithmetic stays on the uniform datapath; a loop run by one lane alone issued at
        // less than half the rate).
        // The products are queued: the warp issues a tile's 25 in a few hundred cycles, the tensor pipe
        // needs 1600 for them.  Everything else this warp sends to shared memory (a look at an mbarrier)
        // is served only after the products queued before it, so a tile has ONE such point, inside the
        // elected block, in the middle of its last k-block: a non-blocking look (test_wait) at all the
        // NEXT tile needs.  When it succeeds, the next tile's products follow this tile's last six with
        // nothing but a vote between them; the blocking wait at the top of a tile runs only when there
        // really is something to wait for (the first tile of a row tile, whose A panels the producers
        // can only write once the previous row tile's last products have retired).
        // What the stream reaches (cycle counters in the issuing warp, this kernel, D = 128, K = 1024):
        // 64 cycles per product when nothing else runs in the CTA (the pipe's own rate), 80 with every
        // role present but idle, 67 of those 80 if the waits on the B ring are left out, 83 with the B
        // copies and the row producers working, 96 with the epilogue's loads and ranking.  A second
        // issuing warp taking every other tile, splitting a tile into more elected blocks, or a fifth
        // ring stage changed none of these figures (three stages cost 17 %); at this rate the B ring
        // draws 7 TB/s from L2.
        {
            constexpr uint32_t IDESC = F16 ? IDESC_F16 : IDESC_TF32;
            const uint64_t desc0 = smem_desc_sw128(smem_u32(st_base));         // stage 0, hi panel, k-step 0
            const uint32_t desc_hi32 = (uint32_t)(desc0 >> 32);
            const uint32_t desc_lo32 = (uint32_t)desc0;
            // K-major, no swizzle: 8-row x 16-byte core matrices, the two k-halves 128 bytes apart
            // (leading byte offset), 8-row groups 256 bytes apart (stride byte offset)
            const uint32_t ext_lo32 = ((smem_u32(st_base + STAGE) & 0x3FFFFu) >> 4) | ((128u >> 4) << 16);
            const uint32_t ext_hi32 = (256u >> 4) | (1u << 14);
            const uint32_t ring = (uint32_t)(p.resident ? nt_count * nkb : NSTAGE);
            struct AccTile {
                int tile, nt;               // row tile, accumulator tile inside it
                uint32_t q;                 // accumulator tiles so far
                uint32_t s, ph;             // B stage of the tile's first k-block and that stage's phase
                uint32_t ab, use, first;    // A buffer, how often it was used before, 1 on the CTA's first row tile
            };
            auto next_stage = [&](uint32_t& st, uint32_t& phase) { if (++st == ring) { st = 0; phase ^= 1u; } };
            auto advance = [&](AccTile& x) {
                for (int kb = 0; kb < nkb; ++kb) next_stage(x.s, x.ph);
                ++x.q;
                if (++x.nt == nt_count) {
                    x.nt = 0; x.tile += stride; x.first = 0u;
                    if (++x.ab == (uint32_t)nab) { x.ab = 0u; ++x.use; }
                }
            };
            // what a tile needs before its first product: its accumulator buffer handed back, (first tile of a
            // row tile) the A panels written, its B stages landed
            auto look = [&](const AccTile& x) -> bool {               // non-blocking, this lane's view
                bool r = mbar_test(BAR(ACC_EMPTY + (x.q & 1u)), ((x.q >> 1) & 1u) ^ 1u);
                uint32_t st = x.s, phase = x.ph;
                for (int kb = 0; kb < nkb; ++kb) {
                    if (x.nt == 0) r = mbar_test(BAR(A_FULL + x.ab * 4 + kb), x.use & 1u) & r;
                    if (!p.resident || x.first) r = mbar_test(BAR(B_FULL + st), phase) & r;
                    next_stage(st, phase);
                }
                return r;
            };
            auto await = [&](const AccTile& x) -> bool {              // bounded waits
                bool r = mbar_wait(BAR(ACC_EMPTY + (x.q & 1u)), ((x.q >> 1) & 1u) ^ 1u, abort_flag);
                uint32_t st = x.s, phase = x.ph;
                for (int kb = 0; kb < nkb && r; ++kb) {
                    if (x.nt == 0) r = mbar_wait(BAR(A_FULL + x.ab * 4 + kb), x.use & 1u, abort_flag);
                    if (r && (!p.resident || x.first)) r = mbar_wait(BAR(B_FULL + st), phase, abort_flag);
                    next_stage(st, phase);
                }
                return __all_sync(0xffffffffu, r);
            };
            AccTile cur = {first, 0, 0u, 0u, 0u, 0u, 0u, 1u};
            bool ready = false;
            while (cur.tile < p.total_tiles && ok) {
                if (!ready) {
                    ok = await(cur);
                    if (!ok) break;
                }
                AccTile nxt = cur;
                advance(nxt);
                const bool has_next = nxt.tile < p.total_tiles;
                const uint32_t a_base = tmem + COL_A + cur.ab * AST;
                const uint32_t d_tmem = tmem + COL_ACC + (cur.q & 1u) * BN;
                bool seen = false;                                   // the elected lane's look at the next tile
                if (elect_one()) {
                    tc_fence_after();
                    uint32_t st = cur.s, phase = cur.ph;
                    for (int kb = 0; kb < nkb; ++kb) {
                        const uint32_t a_hi = a_base + kb * 32, a_lo = a_hi + DC;
                        const uint32_t blo = desc_lo32 + st * (SLOT >> 4);            // this stage's hi panel
                        // The very first product of an accumulator tile overwrites it.  fp16 split: that is
                        // the constant-term product (the row's 16 extra features against the centroid
                        // tile's, which sit behind the first k-block's panels without swizzle).
                        if (F16 && kb == 0)
                            tc_mma_ts<F16>(d_tmem, a_base + 2 * DC, mk_desc(ext_lo32 + st * (SLOT >> 4), ext_hi32), IDESC, 0u);
                        tc_mma_ts<F16>(d_tmem, a_lo, mk_desc(blo, desc_hi32), IDESC, (F16 || kb != 0) ? 1u : 0u);
                        tc_mma_ts_acc<F16>(d_tmem, a_hi, mk_desc(blo + (PANEL >> 4), desc_hi32), IDESC);
                        tc_mma_ts_acc<F16>(d_tmem, a_hi, mk_desc(blo, desc_hi32), IDESC);
                        tc_mma_ts_acc<F16>(d_tmem, a_lo + 8, mk_desc(blo + 2, desc_hi32), IDESC);
                        tc_mma_ts_acc<F16>(d_tmem, a_hi + 8, mk_desc(blo + (PANEL >> 4) + 2, desc_hi32), IDESC);
                        tc_mma_ts_acc<F16>(d_tmem, a_hi + 8, mk_desc(blo + 2, desc_hi32), IDESC);
                        if (kb == nkb - 1 && has_next) {
                            seen = look(nxt);
                            tc_fence_after();
                        }
#pragma unroll
                        for (int k8 = 2; k8 < KBF / 8; ++k8) {
                            tc_mma_ts_acc<F16>(d_tmem, a_lo + k8 * 8, mk_desc(blo + k8 * 2, desc_hi32), IDESC);
                            tc_mma_ts_acc<F16>(d_tmem, a_hi + k8 * 8, mk_desc(blo + (PANEL >> 4) + k8 * 2, desc_hi32), IDESC);
                            tc_mma_ts_acc<F16>(d_tmem, a_hi + k8 * 8, mk_desc(blo + k8 * 2, desc_hi32), IDESC);
                        }
                        if (!p.resident) tc_commit(BAR(B_EMPTY + st));                 // stage reusable once these MMAs retire
                        if (cur.nt == nt_count - 1) tc_commit(BAR(A_EMPTY + cur.ab * 4 + kb));   // A panel reusable
                        if (kb == nkb - 1) tc_commit(BAR(ACC_FULL + (cur.q & 1u)));    // accumulator tile complete
                        next_stage(st, phase);
                    }
                }
                ready = __any_sync(0xffffffffu, seen);
                cur = nxt;
            }
        }
    } else if (warp == 13) {
        // ============================ B loader ========================================
        if (lane == 0 && !(p.absent_b_loader && blockIdx.x == 0)) {
            uint32_t s = 0, ph = 0;
            uint32_t issued = 0;
            for (int tile = first; tile < p.total_tiles && ok; tile += stride) {
                if (p.resident && tile != first) break;            // one pass fills the ring for good
                const int b = tile / p.tiles_per_inst;
                const unsigned char* src = p.bimg + (size_t)b * nt_count * nkb * STAGE;
                for (int i = 0; i < nt_count * nkb; ++i) {
                    ok = mbar_wait(BAR(B_EMPTY + s), ph ^ 1u, abort_flag);
                    if (!ok) break;
                    const bool with_ext = F16 && (i % nkb == 0);   // a tile's first k-block brings its constant terms
                    mbar_expect_tx(BAR(B_FULL + s), with_ext ? STAGE + EXT : STAGE);
                    bulk_g2s(smem_u32(st_base + (size_t)s * SLOT), src + (size_t)i * STAGE, STAGE, BAR(B_FULL + s));
                    if (with_ext)
                        bulk_g2s(smem_u32(st_base + (size_t)s * SLOT + STAGE),
                                 p.bext + ((size_t)b * nt_count + i / nkb) * EXT, EXT, BAR(B_FULL + s));
                    ++issued;
                    if (++s == NSTAGE) { s = 0; ph ^= 1u; }
                }
            }
            if (!ok) {
                // let copies that are still in flight land before the CTA's shared memory goes away
                const uint32_t pending = issued < NSTAGE ? issued : NSTAGE;
                for (uint32_t k = 0; k < pending; ++k) {
                    const uint32_t idx = issued - 1 - k;
                    const uint32_t st = idx % NSTAGE, par = (idx / NSTAGE) & 1u;
                    for (uint32_t i = 0; i < WAIT_LIMIT && !mbar_try(BAR(B_FULL + st), par); ++i) {}
                }
            }
        }
    }

    else if (APRE) {
        // ============================ A loader (pre-split image) ======================
        if (lane == 0) {
            uint32_t issued = 0;
            int it = 0;
            for (int tile = first; tile < p.total_tiles && ok; tile += stride, ++it) {
                const int buf = it % p.nxb;
                ok = mbar_wait(BAR(AS_EMPTY + buf), (uint32_t)(((it / p.nxb) & 1) ^ 1), abort_flag);
                if (!ok) break;
                mbar_expect_tx(BAR(X_FULL + buf), (uint32_t)(ABUF + AINFO));
                bulk_g2s_stream(smem_u32(as_base + (size_t)buf * ABUF), p.aimg + (size_t)tile * ABUF, (uint32_t)ABUF, BAR(X_FULL + buf));
                bulk_g2s(smem_u32(as_info + (size_t)buf * BM * 2), p.ainfo + (size_t)tile * BM * 2, AINFO, BAR(X_FULL + buf));
                ++issued;
            }
            if (!ok) {
                // let copies that are still in flight land before the CTA's shared memory goes away
                const uint32_t nb = (uint32_t)p.nxb, pending = issued < nb ? issued : nb;
                for (uint32_t k = 0; k < pending; ++k) {
                    const uint32_t idx = issued - 1 - k;
                    for (uint32_t i = 0; i < WAIT_LIMIT && !mbar_try(BAR(X_FULL + idx % nb), (idx / nb) & 1u); ++i) {}
                }
            }
        }
    }

    // ---- teardown: every role arrives here, on success or abort ----------------------
    tc_fence_before();
    __syncthreads();
    if (warp == 12) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(TMEM_COLS) : "memory");
    }
    if (tid == 0 && *abort_flag) atomicOr(p.dev_status, STATUS_TIMEOUT);
}

// ---- exact re-evaluation of queued rows (direct form) ------------------------------------
// Two candidates: one warp per row compares the best and the runner-up of the ranking.
// (Called by every block of the fix-up kernel; a label is touched by exactly one warp.)
__device__ __forceinline__ void
fixup_pairs(int nblocks, int N, int D, int K, const float* __restrict__ z, const float* __restrict__ cent,
            const int* __restrict__ flag_count, const int2* __restrict__ pair_rows, int32_t* __restrict__ labels) {
    const int total = flag_count[0];
    const int lane = threadIdx.x & 31;
    const int wpb = blockDim.x >> 5;
    for (int e = blockIdx.x * wpb + (threadIdx.x >> 5); e < total; e += nblocks * wpb) {
        const int2 ent = pair_rows[e];
        const size_t flat = (size_t)ent.x;
        const int b = (int)(flat / N);
        const int a1 = labels[flat], a2 = ent.y;
        const float4* x4 = reinterpret_cast<const float4*>(z + flat * D);
        const float4* c1 = reinterpret_cast<const float4*>(cent + ((size_t)b * K + a1) * D);
        const float4* c2 = reinterpret_cast<const float4*>(cent + ((size_t)b * K + a2) * D);
        float d1 = 0.f, d2 = 0.f;
        for (int q = lane; q < D / 4; q += 32) {
            const float4 x = __ldg(x4 + q), u = __ldg(c1 + q), v = __ldg(c2 + q);
            float e0 = x.x - u.x, e1 = x.y - u.y, e2 = x.z - u.z, e3 = x.w - u.w;
            d1 = fmaf(e0, e0, d1); d1 = fmaf(e1, e1, d1); d1 = fmaf(e2, e2, d1); d1 = fmaf(e3, e3, d1);
            e0 = x.x - v.x; e1 = x.y - v.y; e2 = x.z - v.z; e3 = x.w - v.w;
            d2 = fmaf(e0, e0, d2); d2 = fmaf(e1, e1, d2); d2 = fmaf(e2, e2, d2); d2 = fmaf(e3, e3, d2);
        }
        d1 = kb_warp_sum(d1);
        d2 = kb_warp_sum(d2);
        if (lane == 0 && (d2 < d1 || (d2 == d1 && a2 < a1))) labels[flat] = a2;
    }
}

// Exact re-evaluation of queued rows against all K centroids.  ROWS queued rows form a group and
// share every centroid read: tiles of FX_T centroids are staged through shared memory with
// coalesced, independent loads, thread t then owns centroid t of the tile (warp-shuffle argmin,
// lowest index on ties).  Few queued rows: ROWS = 1, so that a row costs one short pass instead of
// the eight-row loop (the kernel's time is then the latency of its slowest block).
constexpr int FX_T = 256;
constexpr int FX_MAXROWS = 8;
template <int ROWS>
__device__ __forceinline__ void
fixup_full(int N, int D, int K, int total, const float* __restrict__ z, const float* __restrict__ cent,
           const int32_t* __restrict__ full_rows, int32_t* __restrict__ labels, float* xrow, float* ctile,
           float (*red_v)[FX_T / 32], int (*red_i)[FX_T / 32], int* s_inst) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    for (int g0 = blockIdx.x * ROWS; g0 < total; g0 += gridDim.x * ROWS) {
        const int nrow = min(ROWS, total - g0);
        __syncthreads();
        for (int e = tid; e < ROWS * (D / 4); e += FX_T) {
            const int r = e / (D / 4), q = e - r * (D / 4);
            // rows past the end of the queue repeat the last one (their result is discarded)
            reinterpret_cast<float4*>(xrow)[e] =
                __ldg(reinterpret_cast<const float4*>(z + (size_t)full_rows[g0 + min(r, nrow - 1)] * D) + q);
        }
        if (tid < ROWS) s_inst[tid] = full_rows[g0 + min(tid, nrow - 1)] / N;
        __syncthreads();
        float best[ROWS];
        int arg[ROWS];
#pragma unroll
        for (int r = 0; r < ROWS; ++r) { best[r] = INFINITY; arg[r] = 0x7fffffff; }
        bool same_inst = true;
#pragma unroll
        for (int r = 1; r < ROWS; ++r) same_inst = same_inst && (s_inst[r] == s_inst[0]);
        if (same_inst) {
            const int CS = D + 4;                                  // 16-byte aligned, conflict-free float4 rows
            const float* cbase = cent + (size_t)s_inst[0] * K * D;
            for (int j0 = 0; j0 < K; j0 += FX_T) {
                const int nc = min(FX_T, K - j0);
                __syncthreads();
                for (int e = tid; e < nc * (D / 4); e += FX_T) {
                    const int jr = e / (D / 4), q = e - jr * (D / 4);
                    *reinterpret_cast<float4*>(ctile + (size_t)jr * CS + 4 * q) =
                        __ldg(reinterpret_cast<const float4*>(cbase + (size_t)(j0 + jr) * D) + q);
                }
                __syncthreads();
                if (tid < nc) {
                    float acc[ROWS];
#pragma unroll
                    for (int r = 0; r < ROWS; ++r) acc[r] = 0.f;
                    const float4* c4 = reinterpret_cast<const float4*>(ctile + (size_t)tid * CS);
                    for (int d = 0; d < D / 4; ++d) {
                        const float4 c = c4[d];
#pragma unroll
                        for (int r = 0; r < ROWS; ++r) {
                            const float4 x = reinterpret_cast<const float4*>(xrow + r * D)[d];
                            float e0 = x.x - c.x, e1 = x.y - c.y, e2 = x.z - c.z, e3 = x.w - c.w;
                            acc[r] = fmaf(e0, e0, acc[r]); acc[r] = fmaf(e1, e1, acc[r]);
                            acc[r] = fmaf(e2, e2, acc[r]); acc[r] = fmaf(e3, e3, acc[r]);
                        }
                    }
#pragma unroll
                    for (int r = 0; r < ROWS; ++r)
                        if (acc[r] < best[r]) { best[r] = acc[r]; arg[r] = j0 + tid; }   // ascending tiles: lowest index on ties
                }
            }
        } else {
            // rows of one group nearly always share an instance; when they do not, each row reads its own
            for (int j = tid; j < K; j += FX_T) {
                float acc[ROWS];
#pragma unroll
                for (int r = 0; r < ROWS; ++r) acc[r] = 0.f;
                for (int d = 0; d < D / 4; ++d) {
#pragma unroll
                    for (int r = 0; r < ROWS; ++r) {
                        const float4 c = __ldg(reinterpret_cast<const float4*>(cent + ((size_t)s_inst[r] * K + j) * D) + d);
                        const float4 x = reinterpret_cast<const float4*>(xrow + r * D)[d];
                        float e0 = x.x - c.x, e1 = x.y - c.y, e2 = x.z - c.z, e3 = x.w - c.w;
                        acc[r] = fmaf(e0, e0, acc[r]); acc[r] = fmaf(e1, e1, acc[r]);
                        acc[r] = fmaf(e2, e2, acc[r]); acc[r] = fmaf(e3, e3, acc[r]);
                    }
                }
#pragma unroll
                for (int r = 0; r < ROWS; ++r)
                    if (acc[r] < best[r]) { best[r] = acc[r]; arg[r] = j; }   // ascending j: lowest index on ties
            }
        }
#pragma unroll
        for (int r = 0; r < ROWS; ++r) {
            float v = best[r];
            int i = arg[r];
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                const float ov = __shfl_xor_sync(0xffffffffu, v, o);
                const int oi = __shfl_xor_sync(0xffffffffu, i, o);
                if (ov < v || (ov == v && oi < i)) { v = ov; i = oi; }
            }
            if (lane == 0) { red_v[r][warp] = v; red_i[r][warp] = i; }
        }
        __syncthreads();
        if (tid < nrow) {
            float bv = INFINITY;
            int bi = 0x7fffffff;
            for (int w = 0; w < FX_T / 32; ++w) {
                const float v = red_v[tid][w];
                const int i = red_i[tid][w];
                if (v < bv || (v == bv && i < bi)) { bv = v; bi = i; }
            }
            labels[full_rows[g0 + tid]] = bi;
        }
    }
}

// The two-candidate rows are settled by warps that need no shared memory, the rows that need all K
// centroids by blocks that stage centroid tiles in shared memory, in groups sized to the queue's
// length.  With few rows in all (both queues are short: a second launch would cost more than it runs)
// one launch does both, one after the other (`pair_rows` non-null); with many rows the pairs get a
// launch of their own at full occupancy.  (Giving each queue its own share of the blocks of one
// launch was slower: fewer blocks then carry more rows through the full re-evaluation.)
__global__ void __launch_bounds__(FX_T)
assign_fixup_pairs_kernel(int N, int D, int K, const float* __restrict__ z, const float* __restrict__ cent,
                          const int* __restrict__ flag_count, const int2* __restrict__ pair_rows,
                          int32_t* __restrict__ labels) {
    kb_grid_dependency_wait();
    fixup_pairs(gridDim.x, N, D, K, z, cent, flag_count, pair_rows, labels);
}

__global__ void __launch_bounds__(FX_T)
assign_fixup_kernel(int N, int D, int K, const float* __restrict__ z, const float* __restrict__ cent,
                    const int* __restrict__ flag_count, const int2* __restrict__ pair_rows,
                    const int32_t* __restrict__ full_rows, int32_t* __restrict__ labels, uint4* __restrict__ zero,
                    size_t zero_n16) {
    kb_grid_dependency_wait();
    // inside a fit: the accumulators of the centroid update that follows are cleared here (one launch fewer)
    for (size_t i = (size_t)blockIdx.x * FX_T + threadIdx.x; i < zero_n16; i += (size_t)gridDim.x * FX_T)
        zero[i] = make_uint4(0u, 0u, 0u, 0u);
    if (pair_rows) fixup_pairs(gridDim.x, N, D, K, z, cent, flag_count, pair_rows, labels);
    extern __shared__ __align__(16) float fx[];            // [FX_MAXROWS][D] rows | [FX_T][D+4] centroid tile
    __shared__ float red_v[FX_MAXROWS][FX_T / 32];
    __shared__ int red_i[FX_MAXROWS][FX_T / 32];
    __shared__ int s_inst[FX_MAXROWS];
    float* xrow = fx;
    float* ctile = fx + FX_MAXROWS * D;
    const int total = flag_count[1];
    if (total <= 0) return;
    const int per_block = (total + gridDim.x - 1) / gridDim.x;     // uniform over the grid
    if (per_block <= 1) fixup_full<1>(N, D, K, total, z, cent, full_rows, labels, xrow, ctile, red_v, red_i, s_inst);
    else if (per_block <= 2) fixup_full<2>(N, D, K, total, z, cent, full_rows, labels, xrow, ctile, red_v, red_i, s_inst);
    else if (per_block <= 4) fixup_full<4>(N, D, K, total, z, cent, full_rows, labels, xrow, ctile, red_v, red_i, s_inst);
    else fixup_full<8>(N, D, K, total, z, cent, full_rows, labels, xrow, ctile, red_v, red_i, s_inst);
}

// ---- dist2 / inertia / representative from final labels (direct form) -------------------
__global__ void __launch_bounds__(256)
assign_finish_kernel(int N, int D, int K, const float* __restrict__ z, const float* __restrict__ cent,
                     const int32_t* __restrict__ labels, float* __restrict__ dist2, double* __restrict__ ws_inertia,
                     unsigned long long* __restrict__ ws_rep) {
    kb_grid_dependency_wait();
    // lanes of a warp cover the float4 columns of a row; when a row needs fewer than 32 lanes several
    // rows share a warp step, and four steps are in flight per lane
    const int b = blockIdx.y;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int vpr = D >> 2;                                      // float4 per row
    const int lpr = vpr >= 32 ? 32 : (32 % vpr == 0 ? vpr : 32); // lanes per row
    const int rpw = 32 / lpr;                                    // rows per warp step
    const int lane_c = lane % lpr, lane_r = lane / lpr;
    const int rows_per_block = (N + gridDim.x - 1) / gridDim.x;
    const int r0 = blockIdx.x * rows_per_block, r1 = min(N, r0 + rows_per_block);
    constexpr int U = 4;
    double local = 0.0;
    const int step = 8 * rpw;                                    // rows per block step
    const int trips = (max(r1 - r0, 0) + U * step - 1) / (U * step);
    for (int it = 0; it < trips; ++it) {
        const int rb = r0 + it * U * step + warp * rpw + lane_r;
        int lab[U];
#pragma unroll
        for (int u = 0; u < U; ++u) lab[u] = __ldg(labels + (size_t)b * N + min(rb + u * step, r1 - 1));
        float acc[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const size_t flat = (size_t)b * N + min(rb + u * step, r1 - 1);
            const float4* x4 = reinterpret_cast<const float4*>(z + flat * D);
            const float4* c4 = reinterpret_cast<const float4*>(cent + ((size_t)b * K + lab[u]) * D);
            float a = 0.f;
            for (int q = lane_c; q < vpr; q += lpr) {
                const float4 x = __ldg(x4 + q), c = __ldg(c4 + q);
                float e0 = x.x - c.x, e1 = x.y - c.y, e2 = x.z - c.z, e3 = x.w - c.w;
                a = fmaf(e0, e0, a); a = fmaf(e1, e1, a); a = fmaf(e2, e2, a); a = fmaf(e3, e3, a);
            }
            acc[u] = a;
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            float a = acc[u];
            for (int o = 1; o < lpr; o <<= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
            const int r = rb + u * step;
            if (lane_c == 0 && r < r1) {
                const size_t flat = (size_t)b * N + r;
                if (dist2) dist2[flat] = a;
                local += (double)a;
                if (ws_rep) {
                    // all rows of a cluster meet in one word: only a key that beats the value seen so far (a
                    // cached, possibly stale, hence larger one) goes to the atomic unit
                    const unsigned long long key = ((unsigned long long)__float_as_uint(a) << 32) | (unsigned)r;
                    unsigned long long* slot = &ws_rep[(size_t)b * K + lab[u]];
                    if (key < __ldca(slot)) atomicMin(slot, key);
                }
            }
        }
    }
    if (ws_inertia) {
        local = kb_warp_sum(local);
        if (lane == 0 && local != 0.0) atomicAdd(&ws_inertia[b], local);
    }
}

// nstage: stage slots kept in shared memory; apre: nxb buffers of pre-split A panels instead of fp32 rows
size_t tc_smem_bytes(int D, int Kpad /* summed over instances */, int nxb, bool f16, int nstage = NSTAGE, bool apre = false) {
    size_t s = 1024;                                       // alignment slack
    s += (size_t)nstage * (f16 ? SLOT_F16 : STAGE);
    s += apre ? (size_t)nxb * ((size_t)BM * a_row_bytes((D + 63) / 64) + AINFO) : (size_t)nxb * BM * (D + 4) * 4;
    s += (f16 ? (size_t)2 * (Kpad / BN) * 4 : (size_t)Kpad * 4) + 4 * BM * 4 + (4 * BM * 5 + 2) * 4;
    s += 48 * 8 + 16;                                      // barriers, TMEM slot, abort flag
    return s;
}

}  // namespace

// Scratch of the tensor path beyond the generic assign scratch:
// B image | centroid norms | queue counter | queue
size_t kb_ws_need_assign_tc(int B, int N, int D, int K) {
    const size_t Kpad = (size_t)(K + BN - 1) / BN * BN;
    return kb_align256(B * Kpad * D * 8) + kb_align256(B * Kpad * 4) + kb_align256(B * Kpad * 32) +
           kb_align256((size_t)B * INST_STRIDE * 4) + 256 + kb_align256((size_t)B * N * 8) + kb_align256((size_t)B * N * 4);
}

// ---- the pre-split image of Z ------------------------------------------------------------
// Bytes of the image (panels, then the row tables) for a matrix the fp16 kernel can take; 0 otherwise.
size_t kb_ws_need_zsplit(int B, int N, int D, int K) {
    if (B < 1 || N < 1 || D % KBF != 0 || D > 128 || K < 128) return 0;
    const size_t tiles = (size_t)B * ((N + BM - 1) / BM), nkb = (D + 63) / 64;
    return kb_align256(tiles * BM * a_row_bytes((int)nkb)) + kb_align256(tiles * AINFO) + 1024;
}

// Shared-memory plan of the pre-split kernel: the B ring only as long as it has to be, then as many
// A buffers as fit (two at least, three at most).  Returns 0 buffers when it does not fit.
static int apre_plan(const kb_ctx* ctx, int B, int D, int Kpad, int* nstage_alloc) {
    const int nkb = (D + 63) / 64;
    const bool resident = B == 1 && (Kpad / BN) * nkb <= NSTAGE;
    *nstage_alloc = resident ? (Kpad / BN) * nkb : NSTAGE;
    for (int nxb = 3; nxb >= 2; --nxb)
        if (tc_smem_bytes(D, Kpad * B, nxb, true, *nstage_alloc, true) <= (size_t)ctx->max_smem_optin) return nxb;
    return 0;
}

// Builds the image of z at `img` (kb_ws_need_zsplit bytes, 1024-byte aligned) and remembers it in the
// context: assignments of exactly this matrix then run from the image until kb_zsplit_forget.
kb_status kb_zsplit_prepare(kb_ctx* ctx, char* img, int B, int N, int D, int K, const float* z) {
    ctx->zs_src = nullptr;
    const int Kpad = (K + BN - 1) / BN * BN;
    int nstage_alloc = 0;
    if (ctx->assign_path == 3 || kb_ws_need_zsplit(B, N, D, K) == 0 || !kb_assign_tc_supported(ctx, B, D, K) ||
        apre_plan(ctx, B, D, Kpad, &nstage_alloc) == 0)
        return KB_OK;                                      // the kernel that splits rows itself will run
    const int tiles_per_inst = (N + BM - 1) / BM, nkb = (D + 63) / 64;
    const size_t tiles = (size_t)B * tiles_per_inst;
    unsigned char* aimg = reinterpret_cast<unsigned char*>(((uintptr_t)img + 1023) & ~(uintptr_t)1023);
    float* ainfo = reinterpret_cast<float*>(aimg + kb_align256(tiles * BM * a_row_bytes(nkb)));
    const int rows_per_block = 8 * (32 / (nkb * 16));      // 8 warps, one or two rows each
    kb_launch(tc_prep_z_f16_kernel, dim3((unsigned)(tiles_per_inst * BM / rows_per_block), B), 256, 0, ctx->stream, N, D, nkb,
              tiles_per_inst, z, aimg, ainfo);
    KB_LAUNCH_CHECK(ctx, "tc_prep_z_f16_kernel");
    ctx->zs_src = z; ctx->zs_B = B; ctx->zs_N = N; ctx->zs_D = D;
    ctx->zs_img = aimg; ctx->zs_info = ainfo;
    return KB_OK;
}
void kb_zsplit_forget(kb_ctx* ctx) { ctx->zs_src = nullptr; }

// what the kernel can run at all
bool kb_assign_tc_supported(const kb_ctx* ctx, int B, int D, int K) {
    if (D % KBF != 0 || D > 128 || K < 1 || K > 8192 || B < 1) return false;
    const long Kpad = (long)(K + BN - 1) / BN * BN;
    if (Kpad * B > 8192) return false;                     // the norms of every instance stay in shared memory
    return tc_smem_bytes(D, (int)(Kpad * B), 1, true) <= (size_t)ctx->max_smem_optin &&
           tc_smem_bytes(D, (int)(Kpad * B), 1, false) <= (size_t)ctx->max_smem_optin;
}
// what the automatic choice sends there: enough centroids to fill an accumulator tile
// and enough rows for the contraction to outweigh the preparation and fix-up launches
bool kb_assign_tc_eligible(const kb_ctx* ctx, int B, int N, int D, int K) {
    return kb_assign_tc_supported(ctx, B, D, K) && K >= 128 && (long long)B * N >= 4096;
}

// Labels through the tensor path.  `ws` points at kb_ws_need_assign_tc bytes.  `approx`
// (nullable) receives the expanded-form squared distance; `flagged` (nullable, device)
// receives the number of rows that went through the exact re-evaluation.
kb_status kb_launch_assign_tc(kb_ctx* ctx, char* ws, int B, int N, int D, int K, const float* z, const float* c,
                              int32_t* labels, float* approx, int* flagged, float eps) {
    const int Kpad = (K + BN - 1) / BN * BN;
    unsigned char* bimg = reinterpret_cast<unsigned char*>(ws);
    float* cnorm = reinterpret_cast<float*>(ws + kb_align256((size_t)B * Kpad * D * 8));
    unsigned char* bext = reinterpret_cast<unsigned char*>(cnorm) + kb_align256((size_t)B * Kpad * 4);
    float* inst = reinterpret_cast<float*>(bext + kb_align256((size_t)B * Kpad * 32));
    int* flag_count = reinterpret_cast<int*>(reinterpret_cast<char*>(inst) + kb_align256((size_t)B * INST_STRIDE * 4));
    int2* pair_rows = reinterpret_cast<int2*>(reinterpret_cast<char*>(flag_count) + 256);
    int32_t* full_rows = reinterpret_cast<int32_t*>(reinterpret_cast<char*>(pair_rows) + kb_align256((size_t)B * N * 8));

    // the split: fp16 hi/lo (kind::f16, 16 features per instruction) unless the tf32 split is forced
    const bool f16 = ctx->assign_path != 3;
    const int nkb = f16 ? (D + 63) / 64 : D / KBF;
    int gprep = 1;
    if (f16) {
        gprep = (Kpad + 7) / 8 < PREP_MAXG ? (Kpad + 7) / 8 : PREP_MAXG;
        kb_launch(tc_prep_f16_kernel, dim3(gprep, B), 256, 0, ctx->stream, K, D, Kpad, nkb, c, bimg, bext, inst, flag_count);
    } else
        kb_launch(tc_prep_kernel, dim3((Kpad + 7) / 8, B), 256, 0, ctx->stream, K, D, Kpad, nkb, c, bimg, cnorm, flag_count);
    KB_LAUNCH_CHECK(ctx, "tc_prep_kernel");

    TcParams p;
    p.B = B; p.N = N; p.D = D; p.K = K; p.Kpad = Kpad;
    p.nkb = nkb;
    p.DC = f16 ? 32 * nkb : D;
    p.gprep = gprep;
    p.tiles_per_inst = (N + BM - 1) / BM;
    p.total_tiles = p.tiles_per_inst * B;
    p.nxb = tc_smem_bytes(D, Kpad * B, 2, f16) <= (size_t)ctx->max_smem_optin ? 2 : 1;
    p.nstage_alloc = NSTAGE;
    p.eps = eps;
    p.resident = (B == 1 && (Kpad / BN) * nkb <= NSTAGE) ? 1 : 0;
    // a pre-split image of exactly this matrix (made by the fit that is calling): multiply out of it
    bool apre = f16 && ctx->zs_src == z && ctx->zs_B == B && ctx->zs_N == N && ctx->zs_D == D;
    if (apre) {
        const int nxb = apre_plan(ctx, B, D, Kpad, &p.nstage_alloc);
        if (nxb == 0) { apre = false; p.nstage_alloc = NSTAGE; }
        else p.nxb = nxb;
    }
    ctx->last_assign_presplit = apre ? 1 : 0;
    p.aimg = apre ? ctx->zs_img : nullptr;
    p.ainfo = apre ? ctx->zs_info : nullptr;
    p.z = z; p.bimg = bimg; p.cnorm = cnorm; p.bext = bext; p.inst = inst; p.labels = labels; p.approx = approx;
    p.flag_count = flag_count; p.pair_rows = pair_rows; p.full_rows = full_rows; p.dev_status = ctx->dev_status;
    p.wait_limit = ctx->dbg_wait_limit ? ctx->dbg_wait_limit : WAIT_LIMIT;
    p.absent_b_loader = ctx->dbg_skip_arrival;
    const size_t smem = tc_smem_bytes(D, Kpad * B, p.nxb, f16, p.nstage_alloc, apre);
    const int grid = p.total_tiles < ctx->sm_count ? p.total_tiles : ctx->sm_count;
    // with few features per row the epilogue's per-column cost is what limits the kernel:
    // track less there and let the (cheap, K*D is small) full re-evaluation settle near-ties
    const bool track2 = f16 || D >= 96;
#define KB_TC_LAUNCH(T2, F, AP)                                                                \
    do {                                                                                       \
        KB_SMEM_OPTIN(ctx, (assign_tc_kernel<T2, F, AP>), smem);                               \
        kb_launch(assign_tc_kernel<T2, F, AP>, grid, AP ? TC_THREADS_APRE : TC_THREADS, smem, ctx->stream, p); \
    } while (0)
    const int tslot = kb_time_begin(ctx, KB_T_ASSIGN_KERNEL);
    if (apre) KB_TC_LAUNCH(true, true, true);
    else if (track2 && f16) KB_TC_LAUNCH(true, true, false);
    else if (track2) KB_TC_LAUNCH(true, false, false);
    else if (f16) KB_TC_LAUNCH(false, true, false);
    else KB_TC_LAUNCH(false, false, false);
#undef KB_TC_LAUNCH
    kb_time_end(ctx, tslot);
    KB_LAUNCH_CHECK(ctx, "assign_tc_kernel");

    const bool one_launch = (long long)B * N <= 524288;     // about five thousand queued rows at most
    if (!one_launch) {
        kb_launch(assign_fixup_pairs_kernel, 8 * ctx->sm_count, FX_T, 0, ctx->stream, N, D, K, z, c, flag_count, pair_rows, labels);
        KB_LAUNCH_CHECK(ctx, "assign_fixup_pairs_kernel");
    }
    const size_t fsmem = (size_t)FX_MAXROWS * D * 4 + (size_t)FX_T * (D + 4) * 4;
    const int fblocks = (int)(((size_t)ctx->max_smem_optin / (fsmem + 2048)) < 1 ? 1 : ((size_t)ctx->max_smem_optin / (fsmem + 2048)));
    KB_SMEM_OPTIN(ctx, assign_fixup_kernel, fsmem);
    kb_launch(assign_fixup_kernel, (fblocks > 4 ? 4 : fblocks) * ctx->sm_count, FX_T, fsmem, ctx->stream, N, D, K, z, c, flag_count,
              one_launch ? pair_rows : static_cast<int2*>(nullptr), full_rows, labels,
              reinterpret_cast<uint4*>(ctx->fit_acc), ctx->fit_acc ? ctx->fit_acc_bytes / 16 : (size_t)0);
    if (ctx->fit_acc) ctx->fit_acc_clean = 1;
    KB_LAUNCH_CHECK(ctx, "assign_fixup_kernel");
    if (flagged) {   // two counters: rows checked against the runner-up, rows re-evaluated against all centroids
        KB_CUDA(ctx, cudaMemcpyAsync(flagged, flag_count, 2 * sizeof(int), cudaMemcpyDeviceToDevice, ctx->stream));
    }
    return KB_OK;
}

kb_status kb_launch_assign_finish(kb_ctx* ctx, int B, int N, int D, int K, const float* z, const float* c,
                                  const int32_t* labels, float* dist2, double* ws_inertia,
                                  unsigned long long* ws_rep) {
    long want = (4L * ctx->sm_count + B - 1) / B;
    long cap = ((long)N + 63) / 64;
    int G = (int)(want > cap ? cap : want);
    if (G < 1) G = 1;
    kb_launch(assign_finish_kernel, dim3(G, B), 256, 0, ctx->stream, N, D, K, z, c, labels, dist2, ws_inertia, ws_rep);
    KB_LAUNCH_CHECK(ctx, "assign_finish_kernel");
    return KB_OK;
}

