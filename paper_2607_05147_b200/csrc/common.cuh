// Shared device helpers for the DSpark sm_100a kernels: PTX wrappers (mbarrier,
// bulk async copy, warp reductions), the counter-based RNG, launch bookkeeping.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>
#include <chrono>

#include "../../include/dspark.h"

namespace dspark {

// ---------------------------------------------------------------------------------
// Geometry of the streamed passes.  A logit row is cut into blocks, one warp each
// (16 B per lane per vector).  The statistics / argmax passes use 4 KB blocks
// (8 vectors per lane), the residual pass 2 KB blocks of each of its two rows.
// Eight blocks form a piece, the unit one bulk async copy brings into one stage.
// ---------------------------------------------------------------------------------
constexpr int kConsumerWarps = 8;
constexpr int kStreamThreads = (kConsumerWarps + 1) * 32;   // + one producer warp
constexpr int kStatVec = 8;                                 // vectors per lane, statistics / argmax
constexpr int kResidVec = 4;                                // vectors per lane and row, residual
constexpr int kStatBlockBytes = kStatVec * 512;             // 4 KB
constexpr int kResidBlockBytes = kResidVec * 512;           // 2 KB
constexpr int kStageBytes = 32768;                          // one pipeline stage in every mode
constexpr int kStages = 2;

// Upper bound on polls of one mbarrier phase before a kernel gives up (each poll may
// itself block for a short hardware-defined time, so this is on the order of a second).
constexpr uint32_t kWaitPollLimit = 1u << 22;

__host__ __device__ inline int blocks_per_row(int V, int elem_bytes, int block_bytes)
{
    long long bytes = (long long)V * elem_bytes;
    return (int)((bytes + block_bytes - 1) / block_bytes);
}

// ---------------------------------------------------------------------------------
// PTX wrappers
// ---------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p)
{
    return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_fence_init()
{
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait: false when the poll limit ran out.
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity, uint32_t limit = kWaitPollLimit)
{
    for (uint32_t i = 0; i < limit; ++i)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}
// 1-D bulk async copy global -> this CTA's shared memory, completion counted on `bar`.
// dst, src 16-byte aligned, bytes a multiple of 16.
__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, uint32_t bytes, uint64_t* bar)
{
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
        ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar))
        : "memory");
}
// The same copy with an L2 eviction-priority hint for the lines it brings in.
__device__ __forceinline__ void bulk_g2s_hint(void* dst, const void* src, uint32_t bytes, uint64_t* bar, uint64_t policy)
{
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
        ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)), "l"(policy)
        : "memory");
}
__device__ __forceinline__ uint64_t l2_policy_evict_first()
{
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ float ex2_approx(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
// Programmatic dependent launch: every kernel of the library is launched so that its CTAs may be
// scheduled as soon as the previous kernel on the stream drains (no explicit early trigger: CTAs
// that arrive early only poll and take issue slots from the kernel they wait for); pdl_wait()
// returns once that kernel has completed and its writes are visible, and must precede any read of
// its results.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// Waits (bounded) until a 64-bit cell in global memory holds `tag`: how the CTAs of a grid learn that CTA 0
// has zeroed the grid's work counters.  The tag is unique per launch (next_launch_tag), so whatever an
// earlier launch or the caller left in the cell cannot be mistaken for it.
__device__ __forceinline__ bool wait_for_tag(const unsigned long long* cell, unsigned long long tag, uint32_t limit = kWaitPollLimit)
{
    for (uint32_t i = 0; i < limit; ++i) {
        unsigned long long v;
        asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(cell) : "memory");
        if (v == tag) return true;
    }
    return false;
}

// Packed pairs of fp32 (sm_100 f32x2 arithmetic: one instruction, two IEEE-rounded results).
__device__ __forceinline__ uint64_t pack2(float a, float b)
{
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(a), "f"(b));
    return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& a, float& b)
{
    asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(v));
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c)
{
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b)
{
    uint64_t d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ uint64_t mul2(uint64_t a, uint64_t b)
{
    uint64_t d;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
// Warp-wide float max in one instruction (sm_100a redux); NaN inputs are ignored.
__device__ __forceinline__ float warp_max_f32(float x)
{
    float y;
    asm volatile("redux.sync.max.f32 %0, %1, 0xffffffff;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float warp_sum_f32(float x)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    return x;
}
__device__ __forceinline__ double warp_sum_f64(double x)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    return x;
}
__device__ __forceinline__ float bf16lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

// ---------------------------------------------------------------------------------
// Philox4x32-10 (Salmon et al., SC'11).  counter = (position, 0, request, 0), key = seed.
// Word 0 -> accept uniform, word 1 -> resample uniform; u = (word >> 8) * 2^-24.
// ---------------------------------------------------------------------------------
__host__ __device__ inline void philox_round(uint32_t& c0, uint32_t& c1, uint32_t& c2, uint32_t& c3,
                                             uint32_t k0, uint32_t k1)
{
    const uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u;
#ifdef __CUDA_ARCH__
    uint32_t hi0 = __umulhi(M0, c0), hi1 = __umulhi(M1, c2);
#else
    uint32_t hi0 = (uint32_t)(((uint64_t)M0 * c0) >> 32), hi1 = (uint32_t)(((uint64_t)M1 * c2) >> 32);
#endif
    uint32_t lo0 = M0 * c0, lo1 = M1 * c2;
    uint32_t n0 = hi1 ^ c1 ^ k0, n2 = hi0 ^ c3 ^ k1;
    c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
}
__host__ __device__ inline void philox_uniforms(uint64_t seed, uint32_t request, uint32_t position,
                                                float& u_accept, float& u_resample)
{
    uint32_t c0 = position, c1 = 0u, c2 = request, c3 = 0u;
    uint32_t k0 = (uint32_t)seed, k1 = (uint32_t)(seed >> 32);
#pragma unroll
    for (int i = 0; i < 10; ++i) {
        philox_round(c0, c1, c2, c3, k0, k1);
        k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
    }
    u_accept = (float)(c0 >> 8) * (1.0f / 16777216.0f);
    u_resample = (float)(c1 >> 8) * (1.0f / 16777216.0f);
}

// ---------------------------------------------------------------------------------
// Host-side launch bookkeeping (per-kernel event timing, error mapping)
// ---------------------------------------------------------------------------------
struct KernelTimerScope {
    KernelTimerScope(int kernel_id, cudaStream_t stream);
    ~KernelTimerScope();
    int slot;
    cudaStream_t stream;
};
int launch_status();   // maps cudaGetLastError() to DSPARK_OK / DSPARK_ERR_CUDA

// Order-preserving 16-bit key of a bf16 pattern (-0 and +0 share a key; NaN is the caller's business) and back.
__device__ __forceinline__ uint32_t bf16_key(uint32_t b)
{
    if (b == 0x8000u) b = 0u;
    return (b & 0x8000u) ? (0xFFFFu - b) : (b | 0x8000u);
}
__device__ __forceinline__ float bf16_key_value(uint32_t k)
{
    const uint32_t b = (k & 0x8000u) ? (k & 0x7FFFu) : (0xFFFFu - k);
    return __uint_as_float(b << 16);
}

// Threshold search of the top-k / top-p truncation run inside the sampling verifier (truncate.cu): writes
// the threshold of every target row to tau_rows (-inf: no cut) and replaces the block sums of the row's
// statistics by the sums over the kept set; the rows themselves are not modified.
// fp32 rows (truncate_f32.cu): the verifier's virtual truncation of every target row, and the in-place form
int truncate_f32_virtual_launch(const void* target, long long stride_elems, int V, const int32_t* row_offsets, int R, int n_rows,
                                const int32_t* top_k, const float* top_p, float temperature, const float* temperatures,
                                float* tau_rows, float2* stats_t, int nblk, int epb, cudaStream_t stream);
int truncate_f32_in_place(void* target, long long stride_elems, int V, const int32_t* row_offsets, int R, int n_rows,
                          const int32_t* top_k, const float* top_p, float temperature, const float* temperatures,
                          float* out_tau, int32_t* out_kept, cudaStream_t stream);
int truncate_virtual_launch(const void* target, long long stride_bytes, int V, const int32_t* row_offsets, int R, int n_rows,
                            const int32_t* top_k, const float* top_p, float temperature, const float* temperatures,
                            float* tau_rows, float2* stats_t, int nblk, int epb, const int32_t* only_flagged,
                            cudaStream_t stream);

// A nonzero 64-bit value no earlier launch of this process used, and that leftover memory will not hold by
// chance: a counter started from a hash of the clock and an address of this process image.
inline unsigned long long next_launch_tag()
{
    static std::atomic<unsigned long long> counter{[] {
        static int anchor;
        unsigned long long x = (unsigned long long)std::chrono::steady_clock::now().time_since_epoch().count();
        x ^= (unsigned long long)(uintptr_t)&anchor * 0x9E3779B97F4A7C15ull;
        x ^= x >> 31; x *= 0xBF58476D1CE4E5B9ull; x ^= x >> 29;
        return x | 1ull;
    }()};
    unsigned long long t = counter.fetch_add(1, std::memory_order_relaxed);
    return t ? t : counter.fetch_add(1, std::memory_order_relaxed);     // 0 is what the cell holds between launches
}

// Launch with programmatic stream serialization (the kernel must call pdl_wait() first).
template <typename... KArgs, typename... Args>
inline void launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream, Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaLaunchKernelEx(&cfg, kernel, args...);
}

}  // namespace dspark
