// dspark_markov_*: the Markov-head sequential draft step (Section 3.1, Eq. sequential-factorization
// and Eq. markov): draft logits of one block position for all requests,
//     logits[r, :] = U_k[r, :] + W1[x_prev[r]] W2          (rank 256),
// followed by one draw per request from softmax(logits / T) and the confidence
//     c[r] = sigmoid(w^T [h_k[r] ; W1[x_prev[r]]])          (Section 3.2.1, Eq. confidence).
//
// The bias is a dense [R,256] x [256,V] contraction, so it runs on the 5th-generation tensor cores,
// but the step as a whole is bound by HBM (base logits in, draft logits out, W2 once), and the kernel
// is organised around keeping those three streams in flight:
//   * a work unit is one 128-row x 128-column tile of the logits; one persistent CTA per SM walks units
//     of ONE row tile (the grid is a multiple of the row-tile count, so CTAs that share a vocabulary
//     tile run side by side and the second reader finds the W2 tile in L2);
//   * the embedding operand W1[x_prev] of that row tile lives in TENSOR MEMORY for the whole launch: the
//     sixteen epilogue warps gather their rows from the table (256-bit loads) and write them with
//     tcgen05.st, lane = row, 128 columns of two bf16;
//   * shared memory holds the pre-packed W2 tile twice (the next vocabulary tile streams in by one 64 KB
//     bulk copy while the current one is multiplied) and three base-logit tiles;
//   * one thread issues tcgen05.mma (M = N = 128, 16 steps of K = 16, A from tensor memory, B through a
//     shared-memory descriptor) into one of two fp32 accumulators in tensor memory;
//   * base-logit tiles arrive by 2-D tensor-map loads; each epilogue warp reads 32 accumulator columns of
//     its lane quarter back (tcgen05.ld), adds them in place, rounds to bf16 and, for a draft step, takes
//     the softmax (or argmax) statistics of the 32 stored values; the finished tile leaves by a
//     tensor-map store.
// The draw is a second, small kernel on those statistics (one CTA per request): no second pass over the
// logits.  It follows the rule of the verifier's bonus draw for a request with no draft position, applied
// to the STORED bf16 logits, so what the drafter samples from is bit for bit the distribution the
// verifier will later read as q.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cstdio>
#include <cstring>
#include <math.h>

#include "common.cuh"

namespace dspark {

constexpr int kRank = 256;                       // r of the low-rank factorization
constexpr int kTileMN = 128;                     // M and N of one MMA tile
constexpr int kTileBytes = kTileMN * kRank * 2;  // 64 KB of bf16: one packed W2 tile
constexpr int kKChunks = kRank / 8;              // 16-byte chunks along K
constexpr int kChunkBytes = kTileMN * 16;        // one K chunk of a tile: 128 columns x 16 B
constexpr int kGroupRows = 8 * kTileMN;          // rows per launch (the grid is cut to a multiple of the row tiles)
constexpr int kEpiWarps = 16;                    // four per tensor-memory lane quarter, 32 columns of a tile each
constexpr int kGemmThreads = (2 + kEpiWarps) * 32; // producer warp, MMA warp, epilogue warps
constexpr int kTmemCols = 512;                   // accumulators: columns 0..255, embedding tile: 256..383, statistics: 384..415

// Packed W2 tile (K-major, no swizzle): element (n, k) of a 128-column x 256 tile lives at
//   (k / 8) * 2048 + (n / 8) * 128 + (n % 8) * 16 + (k % 8) * 2   bytes,
// i.e. 8 x 16 B core matrices, 16 of them per K chunk.
__host__ __device__ inline size_t packed_offset(int n, int k)
{
    return (size_t)(k >> 3) * kChunkBytes + (size_t)(n >> 3) * 128 + (size_t)(n & 7) * 16 + (size_t)(k & 7) * 2;
}

struct MarkovParams {
    const unsigned char* U; long long u_stride_bytes;
    const unsigned char* W1;                  // [V, 256] bf16
    const unsigned char* W2p;                 // packed tiles
    const int32_t* x_prev;
    int R, V, n_tiles, m_tiles;               // for the GEMM: rows and row tiles of this launch's group
    const unsigned char* H; long long h_stride_bytes; int d;
    const float* w_conf;
    unsigned char* out; long long out_stride_bytes;
    float* out_conf;
    int32_t* dev_status;
    float2* stats;                            // workspace: per (row, vocabulary tile) statistics of the stored logits
    float scale2;                             // log2(e) / T
    float2* out_row_stats; long long row_stats_stride;   // optional: (reference, sum) of every stored row for the verifier
    int l2_hints;                             // 1: keep W2 in L2, stream the logits through it (small launches only)
};

// ---- one-time packing of W2 [256, V] into per-tile K-major blobs ---------------------------------
__global__ void markov_pack_w2_kernel(const __nv_bfloat16* __restrict__ W2, int V, int n_tiles, unsigned char* W2p)
{
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;      // (n, kc)
    const long long total = (long long)n_tiles * kTileMN * kKChunks;
    if (idx >= total) return;
    const int kc = (int)(idx % kKChunks);
    const long long n = idx / kKChunks;                                         // global column
    const int tile = (int)(n / kTileMN), nn = (int)(n % kTileMN);
    __align__(16) __nv_bfloat16 v[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = n < V ? W2[(size_t)(kc * 8 + i) * V + n] : __float2bfloat16(0.f);
    *reinterpret_cast<uint4*>(W2p + (size_t)tile * kTileBytes + packed_offset(nn, kc * 8)) = *reinterpret_cast<uint4*>(v);
}

// ---- confidence head: c = sigmoid(w . [h ; W1[x_prev]]), one CTA per request ---------------------------
// Every thread takes a strided share of the d + 256 products (a handful each, fp32 multiply-adds), the
// warp adds its threads' shares; the caller adds the warps' shares after a __syncthreads and applies
// the sigmoid.  The fp32 rounding of the ~1300 terms stays two orders below the 1e-6 bar on c.
__device__ __forceinline__ float confidence_warp_share(const MarkovParams& P, int r)
{
    const int tid = threadIdx.x;
    const int x = P.x_prev[r];
    float z = 0.f;
    const __nv_bfloat16* h = reinterpret_cast<const __nv_bfloat16*>(P.H + (long long)r * P.h_stride_bytes);
    for (int i = tid; i < P.d; i += blockDim.x) z = fmaf(P.w_conf[i], __bfloat162float(h[i]), z);
    if (x >= 0 && x < P.V) {
        const __nv_bfloat16* e = reinterpret_cast<const __nv_bfloat16*>(P.W1) + (size_t)x * kRank;
        for (int i = tid; i < kRank; i += blockDim.x) z = fmaf(P.w_conf[P.d + i], __bfloat162float(e[i]), z);
    }
    return warp_sum_f32(z);
}
__device__ __forceinline__ float sigmoid_of_shares(const float* s_part, int nwarp)
{
    double z = 0.0;
    for (int w = 0; w < nwarp; ++w) z += (double)s_part[w];
    return 1.f / (1.f + expf(-(float)z));
}

__global__ void __launch_bounds__(256) markov_confidence_kernel(MarkovParams P)
{
    __shared__ float s_part[8];
    pdl_wait();
    const float z = confidence_warp_share(P, blockIdx.x);
    if ((threadIdx.x & 31) == 0) s_part[threadIdx.x >> 5] = z;
    __syncthreads();
    if (threadIdx.x == 0) P.out_conf[blockIdx.x] = sigmoid_of_shares(s_part, 8);
}

// ---- tcgen05 helpers --------------------------------------------------------------------------------
__device__ __forceinline__ uint64_t smem_desc_kmajor(uint32_t smem_addr)
{
    // start address, leading byte offset (between the two 16 B K chunks of one MMA) = 2048,
    // stride byte offset (between 8-column groups) = 128, descriptor version 1, no swizzle
    return (uint64_t)((smem_addr & 0x3FFFFu) >> 4) | ((uint64_t)(kChunkBytes >> 4) << 16) |
           ((uint64_t)(128 >> 4) << 32) | (1ull << 46);
}
// D fp32, A and B bf16, both K-major, N = 128, M = 128
constexpr uint32_t kInstrDesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kTileMN >> 3) << 17) |
                                ((uint32_t)(kTileMN >> 4) << 24);

// D[tmem] (+)= A[tmem] * B[smem descriptor]
__device__ __forceinline__ void umma_bf16_ts(uint32_t tmem_d, uint32_t tmem_a, uint64_t b_desc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(tmem_d), "r"(tmem_a), "l"(b_desc), "r"(kInstrDesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void umma_commit(uint64_t* bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// 32 consecutive fp32 columns of this thread's lane
__device__ __forceinline__ void tmem_load32(uint32_t taddr, float (&v)[32])
{
    uint32_t r[32];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
        "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];\n\t"
        "tcgen05.wait::ld.sync.aligned;"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tmem_store32(uint32_t taddr, const uint4 (&w)[8])
{
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,"
        "%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};"
        ::"r"(taddr), "r"(w[0].x), "r"(w[0].y), "r"(w[0].z), "r"(w[0].w), "r"(w[1].x), "r"(w[1].y), "r"(w[1].z), "r"(w[1].w),
          "r"(w[2].x), "r"(w[2].y), "r"(w[2].z), "r"(w[2].w), "r"(w[3].x), "r"(w[3].y), "r"(w[3].z), "r"(w[3].w),
          "r"(w[4].x), "r"(w[4].y), "r"(w[4].z), "r"(w[4].w), "r"(w[5].x), "r"(w[5].y), "r"(w[5].z), "r"(w[5].w),
          "r"(w[6].x), "r"(w[6].y), "r"(w[6].z), "r"(w[6].w), "r"(w[7].x), "r"(w[7].y), "r"(w[7].z), "r"(w[7].w)
        : "memory");
}

// two / eight consecutive 32-bit columns of this thread's lane
__device__ __forceinline__ void tmem_store2(uint32_t taddr, uint32_t a, uint32_t b)
{
    asm volatile("tcgen05.st.sync.aligned.32x32b.x2.b32 [%0], {%1, %2};\n\ttcgen05.wait::st.sync.aligned;"
                 ::"r"(taddr), "r"(a), "r"(b) : "memory");
}
__device__ __forceinline__ void tmem_load8(uint32_t taddr, uint32_t (&r)[8])
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];\n\ttcgen05.wait::ld.sync.aligned;"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                 : "r"(taddr) : "memory");
}

// A quarter row of an embedding tile: 128 B of W1[x_prev] (src; NULL = zeros) into registers by four
// 256-bit loads (a full 32 B sector each, all in flight at once), then into this thread's lane of tensor
// memory, 32 columns from taddr (two bf16 per column, k ascending).
__device__ __forceinline__ void embedding_quarter_row_load(const unsigned char* src, uint4 (&w)[8])
{
#pragma unroll
    for (int v = 0; v < 8; ++v) w[v] = make_uint4(0, 0, 0, 0);
    if (src)
#pragma unroll
        for (int v = 0; v < 8; v += 2)
            asm volatile("ld.global.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                         : "=r"(w[v].x), "=r"(w[v].y), "=r"(w[v].z), "=r"(w[v].w),
                           "=r"(w[v + 1].x), "=r"(w[v + 1].y), "=r"(w[v + 1].z), "=r"(w[v + 1].w)
                         : "l"(src + v * 16)
                         : "memory");
}
__device__ __forceinline__ void embedding_quarter_row_store(uint32_t taddr, const uint4 (&w)[8])
{
    tmem_store32(taddr, w);
    asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
    tc_fence_before();
}

// ---- 2-D tensor-map copies of the base-logit / output tiles ---------------------------------------
// One box is 64 columns x 128 rows of bf16 (128 B x 128) in the 128-byte swizzle: the 16 B chunk j of
// row r sits at chunk position j ^ (r & 7), so a thread that owns one row reads its chunks without
// bank conflicts against the seven neighbouring rows.
constexpr int kBoxCols = 64;
constexpr int kBoxBytes = kBoxCols * 2 * kTileMN;      // 16 KB
constexpr int kUTileBytes = 2 * kBoxBytes;             // 128 x 128 bf16
constexpr int kUBuffers = 3;

// Both carry an L2 eviction-priority hint.  When one launch's base and draft logits together with the packed
// W2 (66 MB at V = 129 280) fit the L2, the logits are marked evict-first and W2 evict-last, and the next draft
// position finds most of W2 still there (R = 64: 18.7 -> 14.8 us per call); larger launches replace the whole
// L2 anyway and measured a few per cent slower with the hints, so they use the normal priority.
__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* map, int x, int y, uint64_t* bar, uint64_t policy)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3}], [%4], %5;"
        ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(smem_u32(bar)), "l"(policy)
        : "memory");
}
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, int x, int y, const void* src, uint64_t policy)
{
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.tile.bulk_group.L2::cache_hint [%0, {%1, %2}], [%3], %4;"
                 ::"l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(smem_u32(src)), "l"(policy)
                 : "memory");
}
__device__ __forceinline__ uint64_t l2_policy_evict_last()
{
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ uint64_t l2_policy_evict_normal()
{
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_normal.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ void bulk_commit_group() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void bulk_wait_group_read() { asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void fence_proxy_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// acc (fp32) + base logits (bf16 pairs) -> bf16 pairs, round to nearest even
__device__ __forceinline__ uint4 add_round(const float* acc, uint4 u)
{
    const uint32_t uw[4] = {u.x, u.y, u.z, u.w};
    uint32_t ow[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const __nv_bfloat162 b2 = __floats2bfloat162_rn(acc[2 * i] + bf16lo(uw[i]), acc[2 * i + 1] + bf16hi(uw[i]));
        ow[i] = *reinterpret_cast<const uint32_t*>(&b2);
    }
    return make_uint4(ow[0], ow[1], ow[2], ow[3]);
}

// ---- per-tile statistics of the stored logits, taken in the epilogue --------------------------------
// One entry per row and 32 columns (four per vocabulary tile, one per epilogue warp of a lane quarter);
// merge_entries() below folds the four into the tile's entry.
// kStats = 1 (sampling): m = max of the 32 stored values of (row, box), s = sum of 2^((x - m) * scale2),
//   i.e. the box's softmax mass relative to its own maximum.  A NaN or +inf element makes s NaN; a tile
//   with no element above -inf has m = -inf, s = 0.
// kStats = 2 (greedy): m = max, s = the bit pattern of the lowest column index that attains it (-1 if
//   nothing exceeds -inf; NaN never wins).
template <int kStats>
struct TileStats {
    float m, s;
    int idx;
    __device__ __forceinline__ void reset() { m = -INFINITY; s = 0.f; idx = -1; }
    // 32 stored values (16 words of two bf16) starting at column `col`; columns >= V do not count
    __device__ __forceinline__ void update(const uint4 (&o)[4], int col, int V, float scale2)
    {
        if (kStats != 0) accumulate(o, col, V, scale2);
    }
    __device__ __forceinline__ void accumulate(const uint4 (&o)[4], int col, int V, float scale2)
    {
        const uint32_t w[16] = {o[0].x, o[0].y, o[0].z, o[0].w, o[1].x, o[1].y, o[1].z, o[1].w,
                                o[2].x, o[2].y, o[2].z, o[2].w, o[3].x, o[3].y, o[3].z, o[3].w};
        const int nvalid = V - col;                         // >= 32 except in the last tile
        if (kStats == 1 && nvalid >= 32 && m == -INFINITY && s == 0.f) {
            // whole box, fresh entry: maximum on packed bf16 pairs (NaN dropped, as fmaxf does), then one
            // packed multiply-add and two exponentials per pair
            __nv_bfloat162 mx = *reinterpret_cast<const __nv_bfloat162*>(&w[0]);
#pragma unroll
            for (int i = 1; i < 16; ++i) mx = __hmax2(mx, *reinterpret_cast<const __nv_bfloat162*>(&w[i]));
            const uint32_t mb = *reinterpret_cast<const uint32_t*>(&mx);
            const float cm = fmaxf(bf16lo(mb), bf16hi(mb));
            if (cm > -INFINITY) {
                const uint64_t sc = pack2(scale2, scale2), no = pack2(-cm * scale2, -cm * scale2);
                uint64_t a = pack2(0.f, 0.f), b = pack2(0.f, 0.f);
#pragma unroll
                for (int i = 0; i < 16; i += 2) {
                    float t0, t1, t2, t3;
                    unpack2(fma2(pack2(bf16lo(w[i]), bf16hi(w[i])), sc, no), t0, t1);
                    unpack2(fma2(pack2(bf16lo(w[i + 1]), bf16hi(w[i + 1])), sc, no), t2, t3);
                    a = add2(a, pack2(ex2_approx(t0), ex2_approx(t1)));
                    b = add2(b, pack2(ex2_approx(t2), ex2_approx(t3)));
                }
                float s0, s1;
                unpack2(add2(a, b), s0, s1);
                s = s0 + s1;
                m = cm;
                return;
            }
        }
        float x[32];
#pragma unroll
        for (int i = 0; i < 16; ++i) { x[2 * i] = bf16lo(w[i]); x[2 * i + 1] = bf16hi(w[i]); }
        if (kStats == 2) {
#pragma unroll
            for (int i = 0; i < 32; ++i)
                if (i < nvalid && x[i] > m) { m = x[i]; idx = col + i; }
            return;
        }
        float cm = -INFINITY;
#pragma unroll
        for (int i = 0; i < 32; ++i)
            if (i < nvalid) cm = fmaxf(cm, x[i]);           // fmaxf drops NaN: it surfaces in the sum below
        const float mn = fmaxf(m, cm);
        if (mn > -INFINITY) {
            const float off = mn * scale2;
            float a0 = 0.f, a1 = 0.f;
#pragma unroll
            for (int i = 0; i < 32; i += 2) {
                if (i < nvalid) a0 += ex2_approx(fmaf(x[i], scale2, -off));
                if (i + 1 < nvalid) a1 += ex2_approx(fmaf(x[i + 1], scale2, -off));
            }
            s = s * ex2_approx((m - mn) * scale2) + (a0 + a1);
            m = mn;
        } else {
#pragma unroll
            for (int i = 0; i < 32; ++i)
                if (i < nvalid && x[i] != x[i]) s = x[i];
        }
    }
    __device__ __forceinline__ float2 result() const { return make_float2(m, kStats == 2 ? __int_as_float(idx) : s); }
};

// The four 32-column entries of one (row, tile), as (m, s) pairs in column order, merged into the entry
// of the 128-column tile.
template <int kStats>
__device__ __forceinline__ float2 merge_entries(const uint32_t (&e)[8], float scale2)
{
    if (kStats == 2) {
        float best = -INFINITY;
        int idx = -1;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float m = __uint_as_float(e[2 * i]);
            const int id = (int)e[2 * i + 1];
            if (id >= 0 && m > best) { best = m; idx = id; }   // earlier columns win ties
        }
        return make_float2(best, __int_as_float(idx));
    }
    float M = -INFINITY;
#pragma unroll
    for (int i = 0; i < 4; ++i) M = fmaxf(M, __uint_as_float(e[2 * i]));
    float S = 0.f;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float m = __uint_as_float(e[2 * i]), s = __uint_as_float(e[2 * i + 1]);
        // a part without mass (m = -inf, s = 0) adds 0; a NaN sum (NaN or +inf element) carries over
        S += (s == 0.f) ? 0.f : s * ex2_approx((m - M) * scale2);
    }
    return make_float2(M, S);
}

// ---- the GEMM: logits = U + W1[x_prev] W2 for one group of rows, bf16 out -----------------------------
// kTma: base-logit tiles and finished tiles move through the tensor maps (ring of three buffers, added
// in place).  Otherwise (a base address or row pitch that breaks the 16-byte rules) the epilogue
// threads load and store their rows directly.
template <bool kTma, int kStats>
__global__ void __launch_bounds__(kGemmThreads, 1)
markov_gemm_kernel(MarkovParams P, const __grid_constant__ CUtensorMap map_u, const __grid_constant__ CUtensorMap map_out)
{
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);   // swizzle atoms: 1 KB
    unsigned char* sU = smem;                               // three base-logit / output tiles
    unsigned char* sB = smem + kUBuffers * kUTileBytes;     // two W2 tiles
    __shared__ __align__(8) uint64_t b_full[2], b_empty[2], a_full[2], acc_full[2], acc_empty[2];
    __shared__ __align__(8) uint64_t u_full[kUBuffers], epi_done, prefetch_issued, gather_issued;
    __shared__ uint32_t s_tmem_base;
    __shared__ int s_abort;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) {
        for (int s = 0; s < 2; ++s) {
            mbar_init(&b_full[s], 1); mbar_init(&b_empty[s], 1);
            mbar_init(&a_full[s], kEpiWarps);
            mbar_init(&acc_full[s], 1); mbar_init(&acc_empty[s], kEpiWarps);
        }
        for (int s = 0; s < kUBuffers; ++s) mbar_init(&u_full[s], 1);
        mbar_init(&epi_done, kEpiWarps);
        mbar_init(&prefetch_issued, 2);
        mbar_init(&gather_issued, kEpiWarps);
        s_abort = 0;
        mbar_fence_init();
    }
    if (warp == 1) {                                        // the whole tensor memory of this SM
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&s_tmem_base)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    // The packed W2 is a weight, not a result of the previous kernel on the stream: the producer starts
    // on it at once; every other role first waits for that kernel (gathered rows, base logits).
    if (warp != 0) pdl_wait();
    const uint32_t tmem_base = s_tmem_base;
    const uint32_t tmem_a0 = tmem_base + 2 * kTileMN;       // this CTA's embedding tile: columns 256 .. 383
    volatile int* abort_flag = &s_abort;
    auto give_up = [&]() { atomicOr(P.dev_status, DSPARK_DEV_TIMEOUT); *abort_flag = 1; };
    // Work unit u = (vocabulary tile u / m_tiles, row tile u % m_tiles); this CTA takes u = blockIdx.x + k * gridDim.x.
    // gridDim.x is a multiple of m_tiles, so the row tile is the same for all of them and only that tile's
    // embeddings are needed (the CTA next door takes the other row tile of the same vocabulary tiles and
    // finds the W2 tile in L2).
    const int n_units = P.n_tiles * P.m_tiles;
    const int my_tiles = (int)blockIdx.x < n_units ? (n_units - 1 - (int)blockIdx.x) / (int)gridDim.x + 1 : 0;
    const int my_mt = (int)blockIdx.x % P.m_tiles;
    auto unit_ntile = [&](int k) { return ((int)blockIdx.x + k * (int)gridDim.x) / P.m_tiles; };

    if (warp == 0) {
        // ---------------- producer: W2 tiles, one ahead ---------------------------------------------------
        if (lane == 0) {
            const uint64_t pol_keep = P.l2_hints ? l2_policy_evict_last() : l2_policy_evict_normal();
            bool told = false;
            if (my_tiles == 0) { mbar_arrive(&prefetch_issued); told = true; }
            int issued = 0;
            for (int k = 0; k < my_tiles && !*abort_flag; ++k) {
                const int bs = k & 1;
                if (!mbar_wait_bounded(&b_empty[bs], ((uint32_t)(k >> 1) & 1u) ^ 1u)) { give_up(); break; }
                // the second tile waits until the loads of the embedding rows have been issued: those small loads
                // would otherwise queue behind it and the first product would start that much later
                if (k == 1 && !mbar_wait_bounded(&gather_issued, 0u)) { give_up(); break; }
                mbar_arrive_expect_tx(&b_full[bs], kTileBytes);
                bulk_g2s_hint(sB + bs * kTileBytes, P.W2p + (size_t)unit_ntile(k) * kTileBytes, kTileBytes, &b_full[bs], pol_keep);
                issued = k + 1;
                if (!told) { mbar_arrive(&prefetch_issued); told = true; }
            }
            if (*abort_flag) {
                // somebody gave up: leave only after the copies already issued have landed (bounded)
                for (int k = issued - 1; k >= 0 && k >= issued - 2; --k) mbar_wait_bounded(&b_full[k & 1], (uint32_t)(k >> 1) & 1u);
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ---------------------------------------------------------------------
        if (lane == 0) {
            for (int k = 0; k < my_tiles && !*abort_flag; ++k) {
                const int s = k & 1;
                const uint32_t ph = (uint32_t)(k >> 1) & 1u;
                bool ok = mbar_wait_bounded(&b_full[s], ph) && mbar_wait_bounded(&acc_empty[s], ph ^ 1u);
                if (ok && k == 0) ok = mbar_wait_bounded(&a_full[0], 0u);            // resident from then on
                if (!ok) { give_up(); break; }
                tc_fence_after();
                const uint32_t b0 = smem_u32(sB + s * kTileBytes);
#pragma unroll
                for (int ks = 0; ks < kRank / 16; ++ks)
                    umma_bf16_ts(tmem_base + (uint32_t)(s * kTileMN), tmem_a0 + (uint32_t)(ks * 8),
                                 smem_desc_kmajor(b0 + ks * 2 * kChunkBytes), ks > 0 ? 1u : 0u);
                umma_commit(&acc_full[s]);                  // the accumulator may be read
                umma_commit(&b_empty[s]);                   // the W2 tile may be overwritten
            }
        }
    } else {
        // ---------------- epilogue: accumulator + base logits -> bf16 ------------------------------------
        // Sixteen warps: four per tensor-memory lane quarter, each owning 32 columns of every tile.  Before
        // the first tile each warp brings one (lane quarter, K quarter) of the embedding tile into tensor
        // memory.
        const int q = warp & 3;                             // TMEM lane quarter this warp may access
        const int chunk = (warp - 2) >> 2;                  // which 32 columns of a tile
        const int c0 = chunk * 32;
        const int trow = q * 32 + lane;                     // row of the tile this thread owns
        const uint32_t lane_base = (uint32_t)(q * 32) << 16;
        const bool leader = kTma && warp == 2 && lane == 0;
        const uint64_t pol_stream = P.l2_hints ? l2_policy_evict_first() : l2_policy_evict_normal();
        int u_issued = 0;                                   // base-logit tiles requested so far (leader)
        auto issue_u_load = [&](int t) {
            const int nt = unit_ntile(t), mt = my_mt;
            u_issued = t + 1;
            unsigned char* dst = sU + (t % kUBuffers) * kUTileBytes;
            mbar_arrive_expect_tx(&u_full[t % kUBuffers], kUTileBytes);
            tma_load_2d(dst, &map_u, nt * kTileMN, mt * kTileMN, &u_full[t % kUBuffers], pol_stream);
            tma_load_2d(dst + kBoxBytes, &map_u, nt * kTileMN + kBoxCols, mt * kTileMN, &u_full[t % kUBuffers], pol_stream);
        };
        // Order of the first requests: the first W2 tile and the first base-logit tile (the copy instructions share
        // the load/store queue with ordinary loads and would wait behind them), then the loads of the embedding
        // rows, then the second tiles: with both tiles of each ahead of them the embedding rows -- which the first
        // product needs -- arrived last, behind 28 MB of prefetch.
        if (leader && my_tiles > 0) issue_u_load(0);
        if (warp == 2 && lane == 0) mbar_arrive(&prefetch_issued);
        mbar_wait_bounded(&prefetch_issued, 0u);            // a limit that runs out only costs the ordering
        if (my_tiles > 0) {
            const int row = my_mt * kTileMN + trow;
            const unsigned char* src = nullptr;             // rows past R and bad tokens: a zero embedding
            if (row < P.R) {
                const int x = P.x_prev[row];
                if (x >= 0 && x < P.V) src = P.W1 + ((size_t)x * kRank + chunk * (kRank / 4)) * 2;
                else if ((int)blockIdx.x < P.m_tiles && chunk == 0) atomicOr(P.dev_status, DSPARK_DEV_BAD_TOKEN);
            }
            uint4 w[8];
            embedding_quarter_row_load(src, w);
            if (lane == 0) mbar_arrive(&gather_issued);     // the loads are on their way: the next tiles may queue behind them
            if (leader && my_tiles > 1) issue_u_load(1);
            embedding_quarter_row_store(tmem_a0 + lane_base + (uint32_t)(chunk * (kRank / 8)), w);
            __syncwarp();
            if (lane == 0) mbar_arrive(&a_full[0]);
        } else if (lane == 0) {
            mbar_arrive(&gather_issued);
        }
        for (int t = 0; t < my_tiles && !*abort_flag; ++t) {
            const int nt = unit_ntile(t), mt = my_mt;
            const int s = t & 1, ub = t % kUBuffers;
            bool ok = mbar_wait_bounded(&acc_full[s], (uint32_t)(t >> 1) & 1u);
            if (kTma) ok = ok && mbar_wait_bounded(&u_full[ub], (uint32_t)(t / kUBuffers) & 1u);
            if (!__all_sync(0xffffffffu, ok)) {
                if (lane == 0) give_up();
                break;
            }
            tc_fence_after();
            const uint32_t acc_addr = tmem_base + lane_base + (uint32_t)(s * kTileMN);
            // Statistics: every warp leaves the (m, s) of its 32 columns in two spare tensor-memory columns of
            // its lanes (four rotating slots of 8 columns from column 384).  The accumulator of tile t can
            // only have been produced after all warps released tile t - 2, i.e. after they wrote that
            // tile's entries: one warp per lane quarter merges them now and stores the tile's entry.
            const uint32_t stat_base = tmem_base + lane_base + (uint32_t)(3 * kTileMN);
            if (kStats && t >= 2 && chunk == ((t - 2) & 3)) {
                uint32_t e[8];
                tmem_load8(stat_base + (uint32_t)(((t - 2) & 3) * 8), e);
                const int row = my_mt * kTileMN + trow;
                if (row < P.R) P.stats[(size_t)row * P.n_tiles + unit_ntile(t - 2)] = merge_entries<kStats>(e, P.scale2);
            }
            TileStats<kStats> ts;
            ts.reset();
            if (kTma) {
                unsigned char* tile = sU + ub * kUTileBytes;
                {
                    float acc[32];
                    tmem_load32(acc_addr + (uint32_t)c0, acc);
                    unsigned char* rowp = tile + (c0 >> 6) * kBoxBytes + trow * 128;
                    const int j0 = (c0 & 63) >> 3;
                    uint4 o[4];
#pragma unroll
                    for (int v4 = 0; v4 < 4; ++v4) {
                        uint4* cell = reinterpret_cast<uint4*>(rowp + (((j0 + v4) ^ (trow & 7)) << 4));
                        o[v4] = add_round(acc + v4 * 8, *cell);
                        *cell = o[v4];
                    }
                    ts.update(o, nt * kTileMN + c0, P.V, P.scale2);
                }
                if (kStats) {
                    const float2 r2 = ts.result();
                    tmem_store2(stat_base + (uint32_t)((t & 3) * 8 + chunk * 2), __float_as_uint(r2.x), __float_as_uint(r2.y));
                }
                tc_fence_before();
                fence_proxy_async_smem();                   // the tile is read next by the copy engine
                __syncwarp();
                if (lane == 0) { mbar_arrive(&acc_empty[s]); mbar_arrive(&epi_done); }
                if (leader) {
                    if (!mbar_wait_bounded(&epi_done, (uint32_t)t & 1u)) {
                        give_up();                          // the loop condition ends every warp's walk
                    } else {
                        tma_store_2d(&map_out, nt * kTileMN, mt * kTileMN, tile, pol_stream);
                        tma_store_2d(&map_out, nt * kTileMN + kBoxCols, mt * kTileMN, tile + kBoxBytes, pol_stream);
                        bulk_commit_group();
                        bulk_wait_group_read<1>();          // the store of tile t-1 has left its buffer
                        if (t + 2 < my_tiles) issue_u_load(t + 2);
                    }
                }
                __syncwarp();
            } else {
                const int row = mt * kTileMN + trow;
                const bool live = row < P.R;
                const unsigned char* urow = P.U + (long long)row * P.u_stride_bytes;
                unsigned char* orow = P.out + (long long)row * P.out_stride_bytes;
                do {
                    float acc[32];
                    tmem_load32(acc_addr + (uint32_t)c0, acc);
                    const int col = nt * kTileMN + c0;
                    if (!live || col >= P.V) break;
                    const unsigned char* up = urow + (long long)col * 2;
                    unsigned char* op = orow + (long long)col * 2;
                    uint4 o[4];
                    if (col + 32 <= P.V && (((uintptr_t)up | (uintptr_t)op) & 15u) == 0) {
#pragma unroll
                        for (int v4 = 0; v4 < 4; ++v4) {
                            o[v4] = add_round(acc + v4 * 8, __ldg((const uint4*)(up + 16 * v4)));
                            *reinterpret_cast<uint4*>(op + 16 * v4) = o[v4];
                        }
                    } else {
                        uint32_t w[16];
#pragma unroll
                        for (int i = 0; i < 32; ++i) {
                            unsigned short b = 0;
                            if (col + i < P.V) {
                                const float u = __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(up)[i]);
                                const __nv_bfloat16 r = __float2bfloat16_rn(acc[i] + u);
                                reinterpret_cast<__nv_bfloat16*>(op)[i] = r;
                                b = *reinterpret_cast<const unsigned short*>(&r);
                            }
                            if (i & 1) w[i >> 1] |= (uint32_t)b << 16; else w[i >> 1] = b;
                        }
#pragma unroll
                        for (int v4 = 0; v4 < 4; ++v4) o[v4] = make_uint4(w[4 * v4], w[4 * v4 + 1], w[4 * v4 + 2], w[4 * v4 + 3]);
                    }
                    ts.update(o, col, P.V, P.scale2);
                } while (false);
                if (kStats) {
                    const float2 r2 = ts.result();
                    tmem_store2(stat_base + (uint32_t)((t & 3) * 8 + chunk * 2), __float_as_uint(r2.x), __float_as_uint(r2.y));
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&acc_empty[s]);
            }
        }
        if (leader) bulk_wait_group_read<0>();              // shared memory stays valid until the stores have read it
        if (leader && *abort_flag) {
            // somebody gave up: the base-logit loads already issued must land before this CTA leaves (bounded);
            // loads are issued for tiles 0, 1 and then t + 2 after tile t
            for (int t = 0; t < my_tiles && t < u_issued; ++t)
                if (t + kUBuffers >= u_issued) mbar_wait_bounded(&u_full[t % kUBuffers], (uint32_t)(t / kUBuffers) & 1u);
        }
    }
    // everyone meets here; the entries of the last two tiles are merged; then the allocating warp returns
    // the tensor memory
    tc_fence_before();
    __syncthreads();
    if (kStats && warp >= 2 && !*abort_flag) {
        tc_fence_after();
        const int chunk = (warp - 2) >> 2;
        const int row = my_mt * kTileMN + (warp & 3) * 32 + lane;
#pragma unroll 1
        for (int t = my_tiles > 2 ? my_tiles - 2 : 0; t < my_tiles; ++t) {
            if (chunk != (t & 3)) continue;
            uint32_t e[8];
            tmem_load8(tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)(3 * kTileMN + (t & 3) * 8), e);
            if (row < P.R) P.stats[(size_t)row * P.n_tiles + unit_ntile(t)] = merge_entries<kStats>(e, P.scale2);
        }
        tc_fence_before();
    }
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
    }
}

// ---- the draw: one token per request from the tile statistics ---------------------------------------
// One CTA of 256 threads per request; thread t owns the `per` consecutive tiles starting at t * per
// (per = tiles per row / 256, rounded up), so thread order is vocabulary order.
// Sampling (greedy == 0): with M the row maximum and z_i = s_i 2^((m_i - M) scale2) the mass of tile i,
// the running sum (within a thread, then across threads) gives the total Z; the token is the smallest v
// whose running sum of 2^((x_v - M) scale2) exceeds u' Z, u' the second uniform of (seed, request,
// position 0): the tile is located on the tile masses, the element inside it on the 128 stored logits of
// that tile.  A row with NaN, +inf or no finite element sets DSPARK_DEV_BAD_ROW and yields -1.
// Greedy: the lowest index of the row maximum; a row with nothing above -inf sets
// DSPARK_DEV_ALL_NEG_INF and yields 0.
// The token just drawn is the previous token of the next draft position: its embedding row (512 B of W1) is
// asked into L2 now, so that the next contraction's gather does not wait for DRAM.  Called by one warp.
__device__ __forceinline__ void prefetch_embedding(const MarkovParams& P, int token, int lane)
{
    if (lane < 4 && token >= 0 && token < P.V)
        asm volatile("prefetch.global.L2 [%0];" ::"l"(P.W1 + (size_t)token * kRank * 2 + lane * 128));
}

constexpr int kDrawThreads = 256;
constexpr int kStatCols = kTileMN;               // columns per statistics entry
constexpr int kDrawPer = 16;                     // entries per thread at most: V <= 256 * 16 * 128
constexpr int kMaxDrawV = kDrawThreads * kDrawPer * kStatCols;

__global__ void __launch_bounds__(kDrawThreads) markov_draw_kernel(MarkovParams P, int greedy, uint64_t seed, int32_t* out_tokens)
{
    __shared__ float s_red[kDrawThreads / 32];
    __shared__ int s_redi[kDrawThreads / 32];
    __shared__ float s_before;
    __shared__ int s_box, s_last, s_bad;
    __shared__ float s_part[kDrawThreads / 32];
    pdl_wait();
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int r = blockIdx.x;
    const int n_box = P.n_tiles;
    const int per = (n_box + kDrawThreads - 1) / kDrawThreads;
    const float2* st = P.stats + (size_t)r * n_box;
    float2 e[kDrawPer];
#pragma unroll
    for (int k = 0; k < kDrawPer; ++k) {
        const int i = tid * per + k;
        e[k] = (k < per && i < n_box) ? st[i] : make_float2(-INFINITY, greedy ? __int_as_float(-1) : 0.f);
    }
    if (tid == 0) { s_box = 0x7fffffff; s_last = -1; s_bad = 0; }
    if (P.out_conf) {                                       // its loads overlap the statistics loads above
        const float zc = confidence_warp_share(P, r);
        if (lane == 0) s_part[warp] = zc;
    }
    __syncthreads();
    if (P.out_conf && tid == 32) P.out_conf[r] = sigmoid_of_shares(s_part, kDrawThreads / 32);
    if (greedy) {
        float best = -INFINITY;
        int bi = 0x7fffffff;
#pragma unroll
        for (int k = 0; k < kDrawPer; ++k) {
            const int idx = __float_as_int(e[k].y);
            if (idx >= 0 && (e[k].x > best || (e[k].x == best && idx < bi))) { best = e[k].x; bi = idx; }
        }
#pragma unroll
        for (int o = 16; o; o >>= 1) {
            const float ob = __shfl_xor_sync(0xffffffffu, best, o);
            const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
            if (ob > best || (ob == best && oi < bi)) { best = ob; bi = oi; }
        }
        if (lane == 0) { s_red[warp] = best; s_redi[warp] = bi; }
        __syncthreads();
        if (tid == 0) {
            for (int w = 1; w < kDrawThreads / 32; ++w)
                if (s_red[w] > best || (s_red[w] == best && s_redi[w] < bi)) { best = s_red[w]; bi = s_redi[w]; }
            if (bi == 0x7fffffff) { atomicOr(P.dev_status, DSPARK_DEV_ALL_NEG_INF); bi = 0; }
            out_tokens[r] = bi;
        }
        if (tid < 32) prefetch_embedding(P, __shfl_sync(0xffffffffu, bi, 0), tid);
        return;
    }
    // row maximum, unusable rows
    float M = -INFINITY;
    bool bad = false;
#pragma unroll
    for (int k = 0; k < kDrawPer; ++k) { M = fmaxf(M, e[k].x); bad |= (e[k].y != e[k].y); }
    M = warp_max_f32(M);
    if (lane == 0) s_red[warp] = M;
    if (bad) s_bad = 1;
    __syncthreads();
#pragma unroll
    for (int w = 0; w < kDrawThreads / 32; ++w) M = fmaxf(M, s_red[w]);
    bad = s_bad || !(M > -INFINITY) || M == INFINITY;
    __syncthreads();                                        // s_red is reused below
    // box masses, running sum inside the thread, exclusive prefix across threads
    const float offM = M * P.scale2;
    float z[kDrawPer];
    float local = 0.f;
#pragma unroll
    for (int k = 0; k < kDrawPer; ++k) {
        z[k] = (!bad && e[k].y > 0.f) ? e[k].y * ex2_approx(fmaf(e[k].x, P.scale2, -offM)) : 0.f;
        local += z[k];
    }
    float inc = local;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const float n = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += n;
    }
    if (lane == 31) s_red[warp] = inc;
    __syncthreads();
    float wbase = 0.f, Z = 0.f;
#pragma unroll
    for (int w = 0; w < kDrawThreads / 32; ++w) { if (w < warp) wbase += s_red[w]; Z += s_red[w]; }
    // the statistics the sampling verifier would compute from this row: reference max * scale (log2 domain) and the sum
    // of 2^(x * scale - reference); a row that cannot be normalised hands out NaN and is reported by the verifier too
    if (tid == 0 && P.out_row_stats) {
        const bool unusable = bad || !(Z > 0.f) || Z == INFINITY;
        P.out_row_stats[(long long)r * P.row_stats_stride] = unusable ? make_float2(NAN, NAN) : make_float2(offM, Z);
    }
    if (bad || !(Z > 0.f) || Z == INFINITY) {
        if (tid == 0) { atomicOr(P.dev_status, DSPARK_DEV_BAD_ROW); out_tokens[r] = -1; }
        return;
    }
    float ua, ur;
    philox_uniforms(seed, (uint32_t)r, 0u, ua, ur);
    const float thr = ur * Z;
    const float excl = wbase + (inc - local);
    // the first box whose inclusive running sum exceeds thr; the last box with mass as a fallback
    {
        float run = excl;
        int mine = 0x7fffffff, lastp = -1;
#pragma unroll
        for (int k = 0; k < kDrawPer; ++k) {
            run += z[k];
            if (z[k] > 0.f) lastp = tid * per + k;
            if (mine == 0x7fffffff && z[k] > 0.f && run > thr) mine = tid * per + k;
        }
        mine = __reduce_min_sync(0xffffffffu, mine);          // one shared-memory atomic per warp
        lastp = __reduce_max_sync(0xffffffffu, lastp);
        if (lane == 0 && mine != 0x7fffffff) atomicMin(&s_box, mine);
        if (lane == 0 && lastp >= 0) atomicMax(&s_last, lastp);
    }
    __syncthreads();
    const int box = s_box != 0x7fffffff ? s_box : s_last;
    const bool found = s_box != 0x7fffffff;
    if (found && box / per == tid) {                        // the owner publishes the sum before its box
        float run = excl;
#pragma unroll
        for (int k = 0; k < kDrawPer; ++k) {
            if (tid * per + k == box) s_before = run;
            run += z[k];
        }
    }
    __syncthreads();
    if (warp != 0) return;
    // inside the tile: four consecutive columns per lane
    const float before = found ? s_before : 0.f;
    const float thr_in = found ? thr : INFINITY;            // rounding left the sum at or below thr: the last token with mass
    const __nv_bfloat16* row = reinterpret_cast<const __nv_bfloat16*>(P.out + (long long)r * P.out_stride_bytes);
    const int c0 = box * kStatCols + lane * 4;
    float ev[4];
    float lsum = 0.f;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        ev[i] = c0 + i < P.V ? ex2_approx(fmaf(__bfloat162float(row[c0 + i]), P.scale2, -offM)) : 0.f;
        lsum += ev[i];
    }
    float linc = lsum;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const float n = __shfl_up_sync(0xffffffffu, linc, o);
        if (lane >= o) linc += n;
    }
    float cum = before + (linc - lsum);
    int tok = -1, lastp = -1;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        cum += ev[i];
        if (ev[i] > 0.f) lastp = c0 + i;
        if (tok < 0 && ev[i] > 0.f && cum > thr_in) tok = c0 + i;
    }
    const unsigned hit = __ballot_sync(0xffffffffu, tok >= 0);
    const unsigned pos = __ballot_sync(0xffffffffu, lastp >= 0);
    int result;
    if (hit) result = __shfl_sync(0xffffffffu, tok, __ffs(hit) - 1);
    else result = pos ? __shfl_sync(0xffffffffu, lastp, 31 - __clz(pos)) : box * kStatCols;
    if (lane == 0) out_tokens[r] = result;
    prefetch_embedding(P, result, lane);
}

struct MarkovWs { size_t stats, trace, total; };
static MarkovWs markov_layout(int R, int V)
{
    auto up = [](size_t x) { return (x + 255) & ~(size_t)255; };
    MarkovWs w;
    size_t o = 0;
    w.stats = o;  o += up((size_t)R * ((V + kTileMN - 1) / kTileMN) * sizeof(float2));
    w.trace = o;
    w.total = o;
    return w;
}

static bool g_gemm_attr_set[64] = {};
static std::atomic<int> g_markov_path{0};   // 0: tensor-map epilogue when the 16-byte rules hold, 1: always direct

// cuTensorMapEncodeTiled through the runtime's driver entry point lookup (no link against the driver)
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
static EncodeTiledFn encode_tiled_fn()
{
    static EncodeTiledFn fn = nullptr;
    static bool looked = false;
    if (!looked) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)p;
        else
            cudaGetLastError();
        looked = true;
    }
    return fn;
}
// bf16 matrix [rows, cols] with a row pitch in bytes, boxes of 64 columns x 128 rows, 128-byte swizzle;
// reads outside the matrix give zeros, writes outside are dropped
static bool make_tile_map(CUtensorMap* map, const void* base, int rows, int cols, long long pitch_bytes)
{
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn || ((uintptr_t)base & 15u) || (pitch_bytes & 15) || pitch_bytes <= 0) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)pitch_bytes};
    const cuuint32_t box[2] = {(cuuint32_t)kBoxCols, (cuuint32_t)kTileMN};
    const cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace dspark

using namespace dspark;

extern "C" {

int dspark_markov_set_epilogue_path(int path)
{
    if (path != 0 && path != 1) return DSPARK_ERR_INVALID_ARG;
    g_markov_path.store(path, std::memory_order_relaxed);
    return DSPARK_OK;
}

size_t dspark_markov_w2_packed_bytes(int V)
{
    if (V < 1) return 0;
    return (size_t)((V + kTileMN - 1) / kTileMN) * kTileBytes;
}

int dspark_markov_pack_w2(const void* W2, int V, void* W2_packed, void* stream)
{
    if (!W2 || !W2_packed || V < 1) return DSPARK_ERR_INVALID_ARG;
    if (((uintptr_t)W2_packed & 15u) != 0) return DSPARK_ERR_ALIGNMENT;
    const int n_tiles = (V + kTileMN - 1) / kTileMN;
    const long long total = (long long)n_tiles * kTileMN * kKChunks;
    markov_pack_w2_kernel<<<(unsigned)((total + 255) / 256), 256, 0, (cudaStream_t)stream>>>(
        (const __nv_bfloat16*)W2, V, n_tiles, (unsigned char*)W2_packed);
    const int rc = launch_status();
    // The contraction starts fetching the packed weights before it waits for the kernel ahead of it on the
    // stream, so they must be complete, not merely enqueued, when this call returns.
    if (rc == DSPARK_OK && cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return launch_status();
    return rc;
}

size_t dspark_markov_workspace_bytes(int R, int V)
{
    if (R < 1 || V < 1) return 0;
    return markov_layout(R, V).total;
}

// one GEMM launch per group of rows; stats_mode 0 none, 1 softmax masses, 2 argmax
static int markov_launch(const void* U, int64_t u_row_stride, const void* W1, const void* W2_packed,
                         const int32_t* x_prev, int R, int V,
                         const void* H, int64_t h_row_stride, int d, const float* w_conf,
                         void* out_logits, int64_t out_row_stride, float* out_conf, int32_t* dev_status,
                         void* workspace, size_t workspace_bytes, cudaStream_t s, int stats_mode, float temperature,
                         MarkovParams* params_out)
{
    if (!U || !W1 || !W2_packed || !x_prev || !out_logits || !dev_status) return DSPARK_ERR_INVALID_ARG;
    if (R < 1 || V < 1 || u_row_stride < V || out_row_stride < V) return DSPARK_ERR_INVALID_ARG;
    if (out_conf && (!H || !w_conf || d < 0 || h_row_stride < d)) return DSPARK_ERR_INVALID_ARG;
    const MarkovWs w = markov_layout(R, V);
    if (!workspace || workspace_bytes < w.total) return DSPARK_ERR_WORKSPACE;
    if ((((uintptr_t)workspace) & 255u) || ((uintptr_t)W2_packed & 15u) || ((uintptr_t)W1 & 31u)) return DSPARK_ERR_ALIGNMENT;
    MarkovParams P;
    P.U = (const unsigned char*)U; P.u_stride_bytes = (long long)u_row_stride * 2;
    P.W1 = (const unsigned char*)W1; P.W2p = (const unsigned char*)W2_packed; P.x_prev = x_prev;
    P.R = R; P.V = V; P.n_tiles = (V + kTileMN - 1) / kTileMN; P.m_tiles = (R + kTileMN - 1) / kTileMN;
    P.H = (const unsigned char*)H; P.h_stride_bytes = (long long)h_row_stride * 2; P.d = d; P.w_conf = w_conf;
    P.out = (unsigned char*)out_logits; P.out_stride_bytes = (long long)out_row_stride * 2;
    P.out_conf = out_conf; P.dev_status = dev_status;
    P.stats = (float2*)((unsigned char*)workspace + w.stats);
    P.l2_hints = 0;
    P.out_row_stats = nullptr; P.row_stats_stride = 0;
    P.scale2 = stats_mode == 1 ? (float)(1.4426950408889634 / (double)temperature) : 0.f;
    if (params_out) *params_out = P;

    int dev = 0, sms = 0, l2_bytes = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    cudaDeviceGetAttribute(&l2_bytes, cudaDevAttrL2CacheSize, dev);
    const int smem_bytes = kUBuffers * kUTileBytes + 2 * kTileBytes + 1024;
    if (!g_gemm_attr_set[dev & 63]) {
        bool ok = true;
        ok = ok && cudaFuncSetAttribute(markov_gemm_kernel<true, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes) == cudaSuccess;
        ok = ok && cudaFuncSetAttribute(markov_gemm_kernel<true, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes) == cudaSuccess;
        ok = ok && cudaFuncSetAttribute(markov_gemm_kernel<true, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes) == cudaSuccess;
        ok = ok && cudaFuncSetAttribute(markov_gemm_kernel<false, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes) == cudaSuccess;
        ok = ok && cudaFuncSetAttribute(markov_gemm_kernel<false, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes) == cudaSuccess;
        ok = ok && cudaFuncSetAttribute(markov_gemm_kernel<false, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes) == cudaSuccess;
        if (!ok) return launch_status();
        g_gemm_attr_set[dev & 63] = true;
    }
    // one launch per group of up to 1024 rows (8 row tiles): W2 is fetched from HBM once per group, the
    // CTAs that share a vocabulary tile run side by side and find it in L2
    for (int r0 = 0; r0 < R; r0 += kGroupRows) {
        MarkovParams G = P;
        G.R = R - r0 < kGroupRows ? R - r0 : kGroupRows;
        G.m_tiles = (G.R + kTileMN - 1) / kTileMN;
        G.U = P.U + (long long)r0 * P.u_stride_bytes;
        G.out = P.out + (long long)r0 * P.out_stride_bytes;
        G.x_prev = P.x_prev + r0;
        G.stats = P.stats + (size_t)r0 * P.n_tiles;
        G.l2_hints = (4.0 * G.R * V + 2.0 * kRank * V) <= 0.8 * (double)l2_bytes;
        CUtensorMap map_u, map_out;
        memset(&map_u, 0, sizeof map_u);
        memset(&map_out, 0, sizeof map_out);
        const bool tma = g_markov_path.load(std::memory_order_relaxed) != 1 && make_tile_map(&map_u, G.U, G.R, V, P.u_stride_bytes) &&
                         make_tile_map(&map_out, G.out, G.R, V, P.out_stride_bytes);
        KernelTimerScope timer(DSPARK_K_MARKOV_GEMM, s);
        const int units = P.n_tiles * G.m_tiles, cap = sms - sms % G.m_tiles;     // a multiple of the row tiles
        const dim3 grid(units < cap ? units : cap), block(kGemmThreads);
        const size_t sm = (size_t)smem_bytes;
        if (tma) {
            if (stats_mode == 0) launch_pdl(markov_gemm_kernel<true, 0>, grid, block, sm, s, G, map_u, map_out);
            else if (stats_mode == 1) launch_pdl(markov_gemm_kernel<true, 1>, grid, block, sm, s, G, map_u, map_out);
            else launch_pdl(markov_gemm_kernel<true, 2>, grid, block, sm, s, G, map_u, map_out);
        } else {
            if (stats_mode == 0) launch_pdl(markov_gemm_kernel<false, 0>, grid, block, sm, s, G, map_u, map_out);
            else if (stats_mode == 1) launch_pdl(markov_gemm_kernel<false, 1>, grid, block, sm, s, G, map_u, map_out);
            else launch_pdl(markov_gemm_kernel<false, 2>, grid, block, sm, s, G, map_u, map_out);
        }
    }
    return launch_status();
}

int dspark_markov_logits(const void* U, int64_t u_row_stride, const void* W1, const void* W2_packed,
                         const int32_t* x_prev, int R, int V,
                         const void* H, int64_t h_row_stride, int d, const float* w_conf,
                         void* out_logits, int64_t out_row_stride, float* out_conf, int32_t* dev_status,
                         void* workspace, size_t workspace_bytes, void* stream)
{
    MarkovParams P;
    const int rc = markov_launch(U, u_row_stride, W1, W2_packed, x_prev, R, V, H, h_row_stride, d, w_conf, out_logits,
                                 out_row_stride, out_conf, dev_status, workspace, workspace_bytes, (cudaStream_t)stream, 0,
                                 1.f, &P);
    if (rc != DSPARK_OK || !out_conf) return rc;
    launch_pdl(markov_confidence_kernel, dim3(R), dim3(256), 0, (cudaStream_t)stream, P);
    return launch_status();
}

static int draft_step_launch(const void* U, int64_t u_row_stride, const void* W1, const void* W2_packed,
                             const int32_t* x_prev, int R, int V,
                             const void* H, int64_t h_row_stride, int d, const float* w_conf,
                             float temperature, uint64_t seed,
                             void* out_logits, int64_t out_row_stride, int32_t* out_tokens, float* out_conf,
                             float* out_row_stats, int64_t row_stats_stride,
                             int32_t* dev_status, void* workspace, size_t workspace_bytes, void* stream);

int dspark_markov_draft_step(const void* U, int64_t u_row_stride, const void* W1, const void* W2_packed,
                             const int32_t* x_prev, int R, int V,
                             const void* H, int64_t h_row_stride, int d, const float* w_conf,
                             float temperature, uint64_t seed,
                             void* out_logits, int64_t out_row_stride, int32_t* out_tokens, float* out_conf,
                             int32_t* dev_status, void* workspace, size_t workspace_bytes, void* stream)
{
    return draft_step_launch(U, u_row_stride, W1, W2_packed, x_prev, R, V, H, h_row_stride, d, w_conf, temperature, seed,
                             out_logits, out_row_stride, out_tokens, out_conf, nullptr, 0, dev_status, workspace,
                             workspace_bytes, stream);
}

int dspark_markov_draft_step_stats(const void* U, int64_t u_row_stride, const void* W1, const void* W2_packed,
                                   const int32_t* x_prev, int R, int V,
                                   const void* H, int64_t h_row_stride, int d, const float* w_conf,
                                   float temperature, uint64_t seed,
                                   void* out_logits, int64_t out_row_stride, int32_t* out_tokens, float* out_conf,
                                   float* out_row_stats, int64_t row_stats_stride,
                                   int32_t* dev_status, void* workspace, size_t workspace_bytes, void* stream)
{
    if (!out_row_stats || row_stats_stride < 1 || !(temperature > 0.f)) return DSPARK_ERR_INVALID_ARG;
    if (((uintptr_t)out_row_stats & 7u) != 0) return DSPARK_ERR_ALIGNMENT;
    return draft_step_launch(U, u_row_stride, W1, W2_packed, x_prev, R, V, H, h_row_stride, d, w_conf, temperature, seed,
                             out_logits, out_row_stride, out_tokens, out_conf, out_row_stats, row_stats_stride, dev_status,
                             workspace, workspace_bytes, stream);
}

static int draft_step_launch(const void* U, int64_t u_row_stride, const void* W1, const void* W2_packed,
                             const int32_t* x_prev, int R, int V,
                             const void* H, int64_t h_row_stride, int d, const float* w_conf,
                             float temperature, uint64_t seed,
                             void* out_logits, int64_t out_row_stride, int32_t* out_tokens, float* out_conf,
                             float* out_row_stats, int64_t row_stats_stride,
                             int32_t* dev_status, void* workspace, size_t workspace_bytes, void* stream)
{
    if (!out_tokens || !(temperature >= 0.f) || isinf(temperature)) return DSPARK_ERR_INVALID_ARG;
    if (V > kMaxDrawV) return DSPARK_ERR_SHAPE;
    const int greedy = temperature == 0.f;
    MarkovParams P;
    const int rc = markov_launch(U, u_row_stride, W1, W2_packed, x_prev, R, V, H, h_row_stride, d, w_conf, out_logits,
                                 out_row_stride, out_conf, dev_status, workspace, workspace_bytes, (cudaStream_t)stream,
                                 greedy ? 2 : 1, temperature, &P);
    if (rc != DSPARK_OK) return rc;
    P.out_row_stats = (float2*)out_row_stats; P.row_stats_stride = row_stats_stride;
    {
        KernelTimerScope timer(DSPARK_K_MARKOV_DRAW, (cudaStream_t)stream);
        launch_pdl(markov_draw_kernel, dim3(R), dim3(kDrawThreads), 0, (cudaStream_t)stream, P, greedy, seed, out_tokens);
    }
    return launch_status();
}

}  // extern "C"
