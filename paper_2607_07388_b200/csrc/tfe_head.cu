// Early-exit prefetch head (paper Sec. 4.4): p_early = softmax(W_pref h), T_early = TopK(p_early).
//
// The only dense contraction of the method: logits[b][v] = sum_j W_pref[v][j] * h[b][j] with
// V ~ 150 k vocabulary rows, d ~ 1 k and a decode batch of B <= 256 hidden states.  W_pref (V*d*2
// bytes, ~311 MB) is read once per call and is what bounds the call (HBM); the arithmetic only
// keeps up on the tensor cores, so the product runs as tcgen05 MMAs:
//
//   tfe_head_gemm_kernel     persistent, one CTA per SM, warp-specialised.  Every CTA owns a
//                            contiguous range of vocabulary rows and walks it in tiles of 128 rows
//                            (the MMA's M); the batch is the MMA's N.  Warp 0 streams W tiles and
//                            the matching k-slice of h through a ring of shared-memory stages with
//                            TMA (128-byte swizzle), warp 1 issues tcgen05.mma (M=128, N=batch
//                            padded to 16, K=16 per instruction, fp32 accumulators in tensor
//                            memory, two accumulators so that a tile's epilogue overlaps the next
//                            tile's MMAs), warps 2-5 read finished accumulators with tcgen05.ld and
//                            store fp32 logits [B][V].  All mbarrier waits are bounded.
//                            The epilogue also leaves, per sequence, what the selection needs so that
//                            it never reads the logits back: the largest logit of every group of 32
//                            vocabulary rows (one warp's rows of one tile), and per (CTA, epilogue
//                            warp) a running maximum with the sum of exp(z - maximum) over the
//                            warp's rows (online softmax).
//   tfe_head_select_kernel   one block per sequence: logsumexp from the per-warp partial sums; the
//                            K-th largest of the 32-row group maxima is a lower bound of the K-th
//                            largest logit, and every logit at or above it lies in a group whose
//                            maximum is at or above it: about K groups of 32 logits are read back
//                            (8 KB of the 600 KB row), ranked (descending logit, equal logits
//                            ascending token id) and the best K become probabilities exp(z - logsumexp).
//
// The fp32 logits [B][V] are still written (they are an output: tfe_head_buffers), but only the
// candidate groups are read again.
#include <cuda.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdint>
#include <cstring>

#include "../../include/tfe.h"

#define HEAD_TILE_M 128             // vocabulary rows per tile (MMA M)
#define HEAD_TILE_K 64              // bf16 elements per stage along d: one 128-byte swizzle row
#define HEAD_UMMA_K 16              // bf16 elements per tcgen05.mma
#define HEAD_MAX_N 256              // batch columns (MMA N)
#ifndef HEAD_EPI_PER_QUARTER
#define HEAD_EPI_PER_QUARTER 2      // epilogue warps per tensor-memory lane quarter
#endif
#define HEAD_EPI_STRIDE (16 * HEAD_EPI_PER_QUARTER)
#define HEAD_THREADS (64 + 128 * HEAD_EPI_PER_QUARTER)   // warp 0 TMA, warp 1 MMA, the rest epilogue
#define HEAD_MAX_STAGES 8
#define HEAD_MAX_K 128              // top-K limit
#define HEAD_SEL_THREADS 512
#define HEAD_WAIT_LIMIT (1u << 22)  // polls of one mbarrier before a wait gives up
#define HEAD_DYN_SMEM (227 * 1024 - 12288)  // dynamic shared memory of the GEMM: the SM's 227 KB minus its static arrays

// device status bits
#define HEAD_ST_TIMEOUT_PRODUCER 1u
#define HEAD_ST_TIMEOUT_MMA 2u
#define HEAD_ST_TIMEOUT_EPILOGUE 4u

namespace {

// ------------------------------------------------------------------ PTX wrappers

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
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
// Bounded wait: gives up after HEAD_WAIT_LIMIT polls or when another role has given up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile uint32_t *abort_flag)
{
    for (uint32_t i = 0; i < HEAD_WAIT_LIMIT; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((i & 1023u) == 1023u && *abort_flag) return false;
    }
    return false;
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int32_t x, int32_t y,
                                            uint64_t hint)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint"
        " [%0], [%1, {%3, %4}], [%2], %5;"
        :
        : "r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(x), "r"(y), "l"(hint)
        : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t cols)
{
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols)
{
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}

// D[tmem] (+)= A[smem] * B[smem]^T, bf16 inputs, fp32 accumulate; issued by one thread.
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        :
        : "r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// The mbarrier receives one arrival when every MMA issued so far by this thread has completed.
__device__ __forceinline__ void umma_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// 16 consecutive fp32 columns of this thread's tensor-memory lane.
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&v)[16])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
          "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory operand descriptor, K-major tile whose rows are 128 bytes (64 bf16) and were
// written by TMA with the 128-byte swizzle: rows 128 B apart, groups of 8 rows 1024 B apart.
// Fields: start address >> 4 [0,14); leading byte offset >> 4 [16,30) (unused with a swizzle,
// 1); stride byte offset >> 4 [32,46) = 64; descriptor version [46,48) = 1; swizzle mode
// [61,64) = 2 (128 bytes).
__device__ __forceinline__ uint64_t umma_desc_sw128(uint32_t smem_addr)
{
    uint64_t d = (uint64_t)((smem_addr & 0x3FFFFu) >> 4);
    d |= (uint64_t)1 << 16;
    d |= (uint64_t)(1024 >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}

// Instruction descriptor of kind::f16: D fp32 (bits [4,6) = 1), A and B bf16 ([7,10) = [10,13) = 1),
// both K-major (bits 15, 16 = 0), N >> 3 at [17,23), M >> 4 at [24,29).
__host__ __device__ constexpr uint32_t umma_idesc_bf16(uint32_t M, uint32_t N)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | ((N >> 3) << 17) | ((M >> 4) << 24);
}

// fp32 -> uint32 whose unsigned order is the float order (NaN sorts above +inf; not produced here)
__device__ __forceinline__ uint32_t orderable(float x)
{
    const uint32_t u = __float_as_uint(x);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float from_orderable(uint32_t k)
{
    return __uint_as_float((k & 0x80000000u) ? (k & 0x7FFFFFFFu) : ~k);
}

// ------------------------------------------------------------------ GEMM

struct HeadGemmParams {
    int32_t V, d, B;
    int32_t N;                      // B rounded up to 16
    int32_t rows_per_cta;           // multiple of 8
    int32_t tail_rows;              // rows_per_cta % 128: rows of every CTA's last, short tile (0: none)
    int32_t stages;
    uint32_t tmem_cols;             // power of two >= 2 N
    float *logits;                  // [B][ld]
    int64_t ld;
    float *group_max;               // [B][4 * gridDim.x]: running maximum of every (CTA, epilogue warp) per sequence
    float *group_sum;               // [B][4 * gridDim.x]: sum of exp(z - that maximum) over the warp's rows
    float *fine_max;                // [B][n_fine]: largest logit of every (CTA, tile, epilogue warp): 32 vocabulary rows
    int32_t n_fine;                 // gridDim.x * tiles_per_cta * 4
    int32_t tiles_per_cta;
    uint32_t *status;
};

__global__ void __launch_bounds__(HEAD_THREADS, 1)
tfe_head_gemm_kernel(const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_w_tail,
                     const __grid_constant__ CUtensorMap map_h, const HeadGemmParams p)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t s_full[HEAD_MAX_STAGES], s_empty[HEAD_MAX_STAGES], s_acc_full[2], s_acc_empty[2];
    __shared__ uint32_t s_tmem_base;
    __shared__ volatile uint32_t s_abort;
    __shared__ float s_gmax[4][HEAD_MAX_N];            // running column maxima of the four epilogue warps
    __shared__ float s_gsum[4][HEAD_MAX_N];            // sums of exp(z - running maximum) over the warps' rows

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const uint32_t stage_bytes = HEAD_TILE_M * 128u + (uint32_t)p.N * 128u;
    const uint32_t smem_base = smem_u32(smem);

    // this CTA's vocabulary rows and tiles
    const int64_t r0 = (int64_t)blockIdx.x * p.rows_per_cta;
    const int64_t r1 = min((int64_t)p.V, r0 + (int64_t)p.rows_per_cta);
    const int32_t n_rows = (int32_t)max((int64_t)0, r1 - r0);
    const int32_t n_tiles = (n_rows + HEAD_TILE_M - 1) / HEAD_TILE_M;
    const int32_t num_kb = p.d / HEAD_TILE_K;

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) { mbar_init(smem_u32(&s_full[s]), 1); mbar_init(smem_u32(&s_empty[s]), 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(smem_u32(&s_acc_full[a]), 1); mbar_init(smem_u32(&s_acc_empty[a]), 4 * HEAD_EPI_PER_QUARTER); }
        s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(smem_u32(&s_tmem_base), p.tmem_cols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = s_tmem_base;
    // Programmatic dependent launch: everything above ran while the kernel before this one on the stream was
    // still draining; its results (the hidden states) are first touched below.  No early trigger for the
    // selection kernel that follows (measured: 69.7 / 78.0 / 104.6 / 159.9 us without, 74.3 / 78.2 / 104.8 /
    // 161.4 us with, for batches of 32 / 64 / 128 / 256); it is launched with the same attribute and waits
    // for this grid before it reads a logit.
    asm volatile("griddepcontrol.wait;" ::: "memory");

    if (warp == 0) {
        // ============================ TMA producer ============================
        if (lane == 0) {
            const uint64_t hint_stream = 0x12F0000000000000ull;     // evict first: W is read once
            const uint64_t hint_keep = 0x14F0000000000000ull;       // evict last: h is read by every tile
            uint32_t stage = 0, phase = 0;
            bool ok = true;
            for (int32_t t = 0; t < n_tiles && ok; ++t) {
                const int32_t valid = min(HEAD_TILE_M, n_rows - t * HEAD_TILE_M);
                // a short last tile is fetched with the short box: only its rows are read
                const bool use_tail = valid < HEAD_TILE_M && valid == p.tail_rows;
                const uint32_t w_bytes = use_tail ? (uint32_t)p.tail_rows * 128u : HEAD_TILE_M * 128u;
                for (int32_t kb = 0; kb < num_kb; ++kb) {
                    if (!mbar_wait(smem_u32(&s_empty[stage]), phase ^ 1u, &s_abort)) {
                        atomicOr(p.status, HEAD_ST_TIMEOUT_PRODUCER);
                        s_abort = 1;
                        ok = false;
                        break;
                    }
                    const uint32_t bar = smem_u32(&s_full[stage]);
                    const uint32_t dst = smem_base + stage * stage_bytes;
                    mbar_expect_tx(bar, w_bytes + (uint32_t)p.N * 128u);
                    // W_pref was re-laid at creation: the 128 x 64 piece of (CTA, tile, k-slice) is 16 contiguous KB
                    const int32_t piece = ((int32_t)blockIdx.x * p.tiles_per_cta + t) * num_kb + kb;
                    tma_load_2d(dst, use_tail ? &map_w_tail : &map_w, bar, 0, piece * HEAD_TILE_M, hint_stream);
                    tma_load_2d(dst + HEAD_TILE_M * 128u, &map_h, bar, kb * HEAD_TILE_K, 0, hint_keep);
                    if (++stage == (uint32_t)p.stages) { stage = 0; phase ^= 1u; }
                }
            }
        }
    } else if (warp == 1) {
        // ============================ MMA issuer ==============================
        if (lane == 0) {
            const uint32_t idesc = umma_idesc_bf16(HEAD_TILE_M, (uint32_t)p.N);
            uint32_t stage = 0, phase = 0;
            bool ok = true;
            for (int32_t t = 0; t < n_tiles && ok; ++t) {
                const uint32_t acc = (uint32_t)t & 1u, acc_phase = ((uint32_t)t >> 1) & 1u;
                if (!mbar_wait(smem_u32(&s_acc_empty[acc]), acc_phase ^ 1u, &s_abort)) {
                    atomicOr(p.status, HEAD_ST_TIMEOUT_MMA);
                    s_abort = 1;
                    break;
                }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + acc * (uint32_t)p.N;
                for (int32_t kb = 0; kb < num_kb; ++kb) {
                    if (!mbar_wait(smem_u32(&s_full[stage]), phase, &s_abort)) {
                        atomicOr(p.status, HEAD_ST_TIMEOUT_MMA);
                        s_abort = 1;
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    const uint32_t a_addr = smem_base + stage * stage_bytes;
                    const uint64_t a_desc = umma_desc_sw128(a_addr);
                    const uint64_t b_desc = umma_desc_sw128(a_addr + HEAD_TILE_M * 128u);
#pragma unroll
                    for (int k = 0; k < HEAD_TILE_K / HEAD_UMMA_K; ++k) {
                        // 16 bf16 = 32 bytes further along the swizzled row: +2 in the address field
                        umma_bf16(d_tmem, a_desc + (uint64_t)(2 * k), b_desc + (uint64_t)(2 * k), idesc,
                                  (kb > 0 || k > 0) ? 1u : 0u);
                    }
                    umma_commit(smem_u32(&s_empty[stage]));         // the stage is free when these MMAs are done
                    if (++stage == (uint32_t)p.stages) { stage = 0; phase ^= 1u; }
                }
                if (ok) umma_commit(smem_u32(&s_acc_full[acc]));    // the accumulator is complete
            }
        }
    } else {
        // ============================ epilogue ================================
        // Two warps share a tensor-memory lane quarter (a warp may only read the lanes 32 * (warp % 4) .. +31) and
        // split its columns: the 16-column chunks alternate between them.
        const uint32_t quarter = (uint32_t)warp & 3u;               // tensor-memory lanes 32*quarter .. +31
        const int32_t c_first = 16 * ((warp - 2) >> 2);             // this warp's chunks: c_first, c_first + HEAD_EPI_STRIDE, ...
        for (int32_t c0 = c_first; c0 < p.N; c0 += HEAD_EPI_STRIDE)
            if (lane < 16) { s_gmax[quarter][c0 + lane] = -INFINITY; s_gsum[quarter][c0 + lane] = 0.f; }
        __syncwarp();
        // 32-row groups of tiles this CTA does not have (the last CTA's range may end early): no logit
        for (int32_t t = n_tiles; t < p.tiles_per_cta; ++t)
            for (int32_t c0 = c_first; c0 < p.N; c0 += HEAD_EPI_STRIDE)
                if (lane < 16 && c0 + lane < p.B)
                    p.fine_max[(int64_t)(c0 + lane) * p.n_fine + ((int64_t)blockIdx.x * p.tiles_per_cta + t) * 4 + quarter] = -INFINITY;
        for (int32_t t = 0; t < n_tiles; ++t) {
            const uint32_t acc = (uint32_t)t & 1u, acc_phase = ((uint32_t)t >> 1) & 1u;
            if (!mbar_wait(smem_u32(&s_acc_full[acc]), acc_phase, &s_abort)) {
                if (lane == 0) atomicOr(p.status, HEAD_ST_TIMEOUT_EPILOGUE);
                s_abort = 1;
                break;
            }
            tc_fence_after();
            const int32_t valid = min(HEAD_TILE_M, n_rows - t * HEAD_TILE_M);
            const int32_t row_in_tile = (int32_t)(quarter * 32u) + lane;
            const int64_t row = r0 + (int64_t)t * HEAD_TILE_M + row_in_tile;
            const uint32_t taddr = tmem_base + ((quarter * 32u) << 16) + acc * (uint32_t)p.N;
            for (int32_t c0 = c_first; c0 < p.N; c0 += HEAD_EPI_STRIDE) {
                uint32_t v[16];
                tmem_ld16(taddr + (uint32_t)c0, v);
                tmem_ld_wait();
                float f[16];
#pragma unroll
                for (int j = 0; j < 16; ++j) f[j] = row_in_tile < valid ? __uint_as_float(v[j]) : -INFINITY;
                if (row_in_tile < valid) {
#pragma unroll
                    for (int j = 0; j < 16; ++j)
                        if (c0 + j < p.B) p.logits[(int64_t)(c0 + j) * p.ld + row] = f[j];
                }
                // Per column: the maximum over the warp's 32 rows (one warp reduction on the order-preserving integer
                // image of the logit), then the sum of exp(z - maximum) as a 24-bit fixed-point integer sum (the warp
                // reduction has no floating-point addition; a term is at most 1, 32 of them stay below 2^30).  Every
                // lane ends with both for all 16 columns: no shuffles to route, nothing through shared memory.
                float gm[16];
                uint32_t gs[16];
#pragma unroll
                for (int j = 0; j < 16; ++j) gm[j] = from_orderable(__reduce_max_sync(0xFFFFFFFFu, orderable(f[j])));
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    const float ev = row_in_tile < valid ? __expf(f[j] - gm[j]) : 0.f;
                    gs[j] = __reduce_add_sync(0xFFFFFFFFu, __float2uint_rn(ev * 16777216.f));
                }
                // lane j folds column c0 + j into the warp's running (maximum, sum) pair: online softmax
                float my_m = -INFINITY;
                uint32_t my_s = 0;
#pragma unroll
                for (int j = 0; j < 16; ++j)
                    if (lane == j) { my_m = gm[j]; my_s = gs[j]; }
                if (lane < 16) {
                    const int32_t c = c0 + lane;
                    if (c < p.B)
                        p.fine_max[(int64_t)c * p.n_fine + ((int64_t)blockIdx.x * p.tiles_per_cta + t) * 4 + quarter] = my_m;
                    if (my_m > -INFINITY) {
                        const float old_ref = s_gmax[quarter][c], new_ref = fmaxf(old_ref, my_m);
                        const float kept = old_ref == -INFINITY ? 0.f : s_gsum[quarter][c] * __expf(old_ref - new_ref);
                        s_gsum[quarter][c] = kept + (float)my_s * (1.f / 16777216.f) * __expf(my_m - new_ref);
                        s_gmax[quarter][c] = new_ref;
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&s_acc_empty[acc]));
        }
        __syncwarp();
        const int32_t groups = 4 * (int32_t)gridDim.x;
        for (int32_t c0 = c_first; c0 < p.N; c0 += HEAD_EPI_STRIDE) {
            const int32_t c = c0 + lane;
            if (lane < 16 && c < p.B) {
                p.group_max[(int64_t)c * groups + 4 * blockIdx.x + quarter] = s_gmax[quarter][c];
                p.group_sum[(int64_t)c * groups + 4 * blockIdx.x + quarter] = s_gsum[quarter][c];
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem_base, p.tmem_cols);
    }
}

// ------------------------------------------------------------------ selection

struct HeadSelParams {
    const float *logits;
    int64_t ld;
    int32_t V, B, K;
    int32_t *out_tokens;            // [B][K]
    float *out_prob;                // [B][K]
    float *out_lse;                 // [B] or nullptr
    const float *group_max;         // [B][groups] from the GEMM's epilogue: running maxima ...
    const float *group_sum;         // ... and sums of exp(z - maximum) of every (CTA, epilogue warp)
    int32_t groups;
    const float *fine_max;          // [B][n_fine]: largest logit of every 32-row group
    int32_t n_fine, tiles_per_cta, rows_per_cta;
};

// Selection, one block per sequence.  Keys are orderable(z) << 32 | ~token -- distinct, so "largest K keys" has
// one answer: descending logit, equal logits ascending token id.
//
// The GEMM's epilogue left the largest logit of every group of 32 vocabulary rows.  The K-th largest of them
// (with multiplicity) bounds the row's K-th largest logit from below (K different logits reach it), and a logit
// at or above the bound sits in a group whose maximum is at or above it: only those groups -- K of them, more
// with equal maxima -- are read back, the logits at or above the bound are kept, each survivor finds its rank
// by counting the survivors above it.  More than HEAD_KEEP_CAP survivors (many equal logits) send the block to
// an exact radix selection over the whole row, eight 8-bit digits, slower but indifferent to the distribution.
// The softmax denominator comes from the epilogue's per-warp (maximum, sum) pairs; no logit is read for it.
#define HEAD_KEEP_CAP 2048
#define HEAD_MAX_FINE 6144

__device__ __forceinline__ unsigned long long head_key(float z, int32_t token)
{
    return ((unsigned long long)orderable(z) << 32) | (uint32_t)~(uint32_t)token;
}

#ifdef HEAD_TIMELINE
__device__ long long g_head_tl[16];
#define HSTAMP(i) do { if (blockIdx.x == 0 && threadIdx.x == 0) g_head_tl[i] = clock64(); } while (0)
#else
#define HSTAMP(i) do { } while (0)
#endif
__global__ void __launch_bounds__(HEAD_SEL_THREADS)
tfe_head_select_kernel(const HeadSelParams p)
{
    __shared__ unsigned long long s_keep[HEAD_KEEP_CAP];
    __shared__ uint32_t s_fine[HEAD_MAX_FINE];
    __shared__ float s_red[HEAD_SEL_THREADS / 32];
    __shared__ uint32_t s_hist[256];
    __shared__ unsigned long long s_prefix;
    __shared__ uint32_t s_want, s_fill, s_nkeep;
    const int b = blockIdx.x;
    const float *row = p.logits + (int64_t)b * p.ld;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    constexpr int NW = HEAD_SEL_THREADS / 32;
    const int32_t G = p.groups;

    // launched with programmatic stream serialisation: the blocks may be resident before the GEMM has
    // finished; nothing of its output is read before this point
    asm volatile("griddepcontrol.wait;" ::: "memory");
    HSTAMP(0);

    // ---- logsumexp from the epilogue's partial sums (at most 2 * HEAD_SEL_THREADS groups: two per thread)
    const float *gmax = p.group_max + (int64_t)b * G, *gsum = p.group_sum + (int64_t)b * G;
    const bool h0 = (int)threadIdx.x < G, h1 = (int)threadIdx.x + HEAD_SEL_THREADS < G;
    const float m0 = h0 ? __ldcg(gmax + threadIdx.x) : -INFINITY, m1 = h1 ? __ldcg(gmax + threadIdx.x + HEAD_SEL_THREADS) : -INFINITY;
    const float t0 = h0 ? __ldcg(gsum + threadIdx.x) : 0.f, t1 = h1 ? __ldcg(gsum + threadIdx.x + HEAD_SEL_THREADS) : 0.f;
    float row_max = fmaxf(m0, m1);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) row_max = fmaxf(row_max, __shfl_xor_sync(0xFFFFFFFFu, row_max, o));
    if (lane == 0) s_red[warp] = row_max;
    if (threadIdx.x == 0) { s_prefix = 0; s_fill = 0; s_nkeep = 0; }
    __syncthreads();
    row_max = s_red[0];
    for (int w = 1; w < NW; ++w) row_max = fmaxf(row_max, s_red[w]);
    __syncthreads();                                // s_red is reused for the sums
    float sum = (t0 > 0.f ? t0 * __expf(m0 - row_max) : 0.f) + (t1 > 0.f ? t1 * __expf(m1 - row_max) : 0.f);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xFFFFFFFFu, sum, o);
    if (lane == 0) s_red[warp] = sum;
    __syncthreads();
    float total = 0.f;
    for (int w = 0; w < NW; ++w) total += s_red[w];
    const float lse = row_max + __logf(total);
    if (threadIdx.x == 0 && p.out_lse) p.out_lse[b] = lse;

    HSTAMP(1);
    // ---- a lower bound of the row's K-th largest logit: the K-th largest (with multiplicity) of the per-(CTA,
    // epilogue warp) maxima, rounded down to the upper 16 bits of its integer image (any lower bound serves):
    // radix selection, two 8-bit digits, most significant first.  With fewer than K such groups: no bound.
    uint32_t theta_key = 0;                         // below every image
    if (G >= p.K) {
        uint32_t prefix = 0, want = (uint32_t)p.K;
        for (int shift = 24; shift >= 16; shift -= 8) {
            if (threadIdx.x < 256) s_hist[threadIdx.x] = 0;
            __syncthreads();
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                const uint32_t gkey = orderable(half ? m1 : m0);
                const bool live = (half ? h1 : h0) && (shift == 24 || (gkey >> (shift + 8)) == (prefix >> (shift + 8)));
                const uint32_t digit = (gkey >> shift) & 255u;
                const uint32_t vote = __ballot_sync(0xFFFFFFFFu, live);
                if (live) {                         // one shared-memory atomic per distinct digit of the warp
                    const uint32_t peers = __match_any_sync(vote, digit);
                    if (lane == __ffs(peers) - 1) atomicAdd(&s_hist[digit], __popc(peers));
                }
            }
            __syncthreads();
            // every warp repeats the search: lane l owns digits 255-8l .. 248-8l, largest first
            uint32_t c[8], local = 0;
#pragma unroll
            for (int j = 0; j < 8; ++j) { c[j] = s_hist[255 - 8 * lane - j]; local += c[j]; }
            uint32_t incl = local;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const uint32_t v = __shfl_up_sync(0xFFFFFFFFu, incl, o);
                if (lane >= o) incl += v;
            }
            const bool owner = incl >= want && incl - local < want;
            uint32_t dgt = 0, rest = 0;
            if (owner) {
                uint32_t before = incl - local;
                int j = 0;
                for (; j < 7 && before + c[j] < want; ++j) before += c[j];
                dgt = 255u - 8u * lane - j;
                rest = want - before;
            }
            const uint32_t who = __ffs(__ballot_sync(0xFFFFFFFFu, owner)) - 1;
            prefix |= __shfl_sync(0xFFFFFFFFu, dgt, who) << shift;
            want = __shfl_sync(0xFFFFFFFFu, rest, who);
            __syncthreads();
        }
        theta_key = prefix;
    }
    HSTAMP(2);

    // ---- the 32-row groups that can hold a logit at or above the bound (their maximum reaches it): a list
    const int32_t F = p.n_fine;
    const float *fmax_row = p.fine_max + (int64_t)b * F;
    {
        constexpr int PER = HEAD_MAX_FINE / HEAD_SEL_THREADS;       // all of a thread's loads in flight together
        float fm[PER];
#pragma unroll
        for (int u = 0; u < PER; ++u) {
            const int32_t g = (int32_t)threadIdx.x + u * HEAD_SEL_THREADS;
            fm[u] = g < F ? __ldcg(fmax_row + g) : -INFINITY;
        }
#pragma unroll
        for (int u = 0; u < PER; ++u) {
            const int32_t g = (int32_t)threadIdx.x + u * HEAD_SEL_THREADS;
            if (g < F && orderable(fm[u]) >= theta_key) {
                const uint32_t at = atomicAdd(&s_fill, 1u);
                if (at < HEAD_MAX_FINE) s_fine[at] = (uint32_t)g;
            }
        }
    }
    __syncthreads();
    HSTAMP(3);
    // ---- read them back, one warp per group, one row per lane, four groups in flight per warp
    const uint32_t n_list = min(s_fill, (uint32_t)HEAD_MAX_FINE);
    for (uint32_t i0 = warp; i0 < n_list; i0 += 4 * NW) {
        float z[4];
        int64_t vv[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const uint32_t i = i0 + (uint32_t)u * NW;
            vv[u] = -1;
            z[u] = 0.f;
            if (i < n_list) {
                const int32_t g = (int32_t)s_fine[i];
                const int32_t cta = g / (4 * p.tiles_per_cta), rest = g - cta * 4 * p.tiles_per_cta;
                const int32_t in_cta = (rest >> 2) * HEAD_TILE_M + (rest & 3) * 32 + lane;
                const int64_t v = (int64_t)cta * p.rows_per_cta + in_cta;
                if (in_cta < p.rows_per_cta && v < p.V) { vv[u] = v; z[u] = __ldcg(row + v); }
            }
        }
#pragma unroll
        for (int u = 0; u < 4; ++u)
            if (vv[u] >= 0 && orderable(z[u]) >= theta_key) {
                const uint32_t at = atomicAdd(&s_nkeep, 1u);
                if (at < HEAD_KEEP_CAP) s_keep[at] = head_key(z[u], (int32_t)vv[u]);
            }
    }
    __syncthreads();
    HSTAMP(4);
    const uint32_t n_keep = s_nkeep;
#ifdef HEAD_TIMELINE
    if (blockIdx.x == 0 && threadIdx.x == 0) g_head_tl[8] = n_keep;
#endif
    const uint32_t take = (uint32_t)min(p.K, p.V);
    if (threadIdx.x == 0) s_want = take;
    if (n_keep <= HEAD_KEEP_CAP) {
        // (fewer survivors than K cannot happen: K logits reach the bound)
        for (uint32_t i = threadIdx.x; i < n_keep; i += blockDim.x) {
            const unsigned long long key = s_keep[i];
            uint32_t rank = 0;
            for (uint32_t j = 0; j < n_keep; ++j) rank += s_keep[j] > key;
            if (rank < take) {
                p.out_tokens[(int64_t)b * p.K + rank] = (int32_t)~(uint32_t)key;
                p.out_prob[(int64_t)b * p.K + rank] = __expf(from_orderable((uint32_t)(key >> 32)) - lse);
            }
        }
    } else {
        // ---- exact radix selection of the row's take-th largest key, most significant byte first
        __syncthreads();
        for (int shift = 56; shift >= 0; shift -= 8) {
            for (int i = threadIdx.x; i < 256; i += blockDim.x) s_hist[i] = 0;
            __syncthreads();
            const unsigned long long prefix = s_prefix;
            for (int i = threadIdx.x; i < p.V; i += blockDim.x) {
                const unsigned long long key = head_key(__ldcg(row + i), i);
                if (shift == 56 || (key >> (shift + 8)) == (prefix >> (shift + 8)))
                    atomicAdd(&s_hist[(uint32_t)(key >> shift) & 255u], 1u);
            }
            __syncthreads();
            if (threadIdx.x == 0) {
                uint32_t want = s_want;
                int dgt = 255;
                for (; dgt > 0 && s_hist[dgt] < want; --dgt) want -= s_hist[dgt];
                s_prefix = prefix | ((unsigned long long)dgt << shift);
                s_want = want;
            }
            __syncthreads();
        }
        // the keys at or above it are exactly `take`; they fit the keep list (take <= HEAD_MAX_K)
        const unsigned long long kth = s_prefix;
        if (threadIdx.x == 0) s_fill = 0;           // (it counted the group list above)
        __syncthreads();
        for (int i = threadIdx.x; i < p.V; i += blockDim.x) {
            const unsigned long long key = head_key(__ldcg(row + i), i);
            if (key >= kth) s_keep[atomicAdd(&s_fill, 1u)] = key;
        }
        __syncthreads();
        for (uint32_t i = threadIdx.x; i < take; i += blockDim.x) {
            const unsigned long long key = s_keep[i];
            uint32_t rank = 0;
            for (uint32_t j = 0; j < take; ++j) rank += s_keep[j] > key;
            p.out_tokens[(int64_t)b * p.K + rank] = (int32_t)~(uint32_t)key;
            p.out_prob[(int64_t)b * p.K + rank] = __expf(from_orderable((uint32_t)(key >> 32)) - lse);
        }
    }
    HSTAMP(5);
}

// ------------------------------------------------------------------ host side

typedef CUresult (*encode_tiled_fn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                    const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                    CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

encode_tiled_fn get_encode_tiled()
{
    static encode_tiled_fn fn = nullptr;
    if (!fn) {
        void *sym = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<encode_tiled_fn>(sym);
    }
    return fn;
}

// W_pref [V][d] row-major -> pieces of 128 rows x 64 columns (16 KB each, rows 128 bytes apart), in the order the
// GEMM's CTAs read them: piece ((cta * tiles_per_cta + tile) * d / 64 + k-slice).  A tile's k-slice is then one
// contiguous 16 KB read instead of 128 reads of 128 bytes 2 * d bytes apart.  Rows a tile does not have are zero.
__global__ void __launch_bounds__(256)
tfe_head_retile_kernel(const uint4 *__restrict__ w, uint4 *__restrict__ tiled, int32_t V, int32_t d, int32_t rows_per_cta,
                       int32_t tiles_per_cta, int64_t n_pieces)
{
    const int32_t num_kb = d / HEAD_TILE_K;
    const int64_t n_vec = n_pieces * HEAD_TILE_M * 8;               // 16-byte vectors: 8 per 128-byte row of a piece
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n_vec; i += (int64_t)gridDim.x * blockDim.x) {
        const int32_t vec = (int32_t)(i & 7), r = (int32_t)((i >> 3) & (HEAD_TILE_M - 1));
        const int64_t piece = i >> 10;
        const int32_t kb = (int32_t)(piece % num_kb);
        const int64_t tile = piece / num_kb;
        const int32_t t = (int32_t)(tile % tiles_per_cta);
        const int64_t cta = tile / tiles_per_cta;
        const int64_t in_cta = (int64_t)t * HEAD_TILE_M + r, row = cta * rows_per_cta + in_cta;
        uint4 v = make_uint4(0, 0, 0, 0);
        if (in_cta < rows_per_cta && row < V) v = w[row * (d / 8) + kb * 8 + vec];
        tiled[i] = v;
    }
}

// bf16 matrix [rows][cols] row-major, box = 64 columns x box_rows rows, 128-byte swizzle
bool make_map(CUtensorMap *map, const void *base, uint64_t rows, uint64_t cols, uint32_t box_rows)
{
    encode_tiled_fn enc = get_encode_tiled();
    if (!enc) return false;
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {cols * 2};
    const cuuint32_t box[2] = {HEAD_TILE_K, box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

struct tfe_head {
    void *d_w_tiled = nullptr;              // W_pref in the GEMM's reading order (tfe_head_retile_kernel)
    int32_t V = 0, d = 0, max_batch = 0;
    int device = 0, sm_count = 0;
    int32_t rows_per_cta = 0, tail_rows = 0, grid = 0;
    CUtensorMap map_w, map_w_tail;
    float *d_logits = nullptr;
    int64_t ld = 0;
    float *d_lse = nullptr;
    uint32_t *d_status = nullptr;
    float *d_group_max = nullptr, *d_group_sum = nullptr, *d_fine_max = nullptr;
    int32_t tiles_per_cta = 0, n_fine = 0;
};

extern "C" {

tfe_status tfe_head_create(const void *w_pref, int32_t V, int32_t d, int32_t max_batch, tfe_head **out)
{
    if (!out) return TFE_ERR_INVALID_ARG;
    *out = nullptr;
    if (!w_pref || V < 1 || d < HEAD_TILE_K || d % HEAD_TILE_K != 0 || max_batch < 1 || max_batch > HEAD_MAX_N)
        return TFE_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(w_pref) & 15u) != 0) return TFE_ERR_INVALID_ARG;
    tfe_head *h = new tfe_head();
    auto fail = [&](tfe_status st) { tfe_head_destroy(h); return st; };
    h->V = V; h->d = d; h->max_batch = max_batch;
    if (cudaGetDevice(&h->device) != cudaSuccess) return fail(TFE_ERR_CUDA);
    if (cudaDeviceGetAttribute(&h->sm_count, cudaDevAttrMultiProcessorCount, h->device) != cudaSuccess)
        return fail(TFE_ERR_CUDA);
    // contiguous row ranges of equal size (a multiple of 8) per CTA
    // (the selection kernel holds at most 2 * HEAD_SEL_THREADS groups = 4 per CTA)
    const int32_t ctas = std::max(1, std::min(std::min(h->sm_count, 2 * HEAD_SEL_THREADS / 4), (V + HEAD_TILE_M - 1) / HEAD_TILE_M));
    h->rows_per_cta = (int32_t)((((int64_t)V + ctas - 1) / ctas + 7) / 8 * 8);
    h->grid = (int32_t)(((int64_t)V + h->rows_per_cta - 1) / h->rows_per_cta);
    h->tail_rows = h->rows_per_cta % HEAD_TILE_M;
    h->ld = ((int64_t)V + 3) / 4 * 4;
    h->tiles_per_cta = (h->rows_per_cta + HEAD_TILE_M - 1) / HEAD_TILE_M;
    {
        const int64_t n_pieces = (int64_t)h->grid * h->tiles_per_cta * (d / HEAD_TILE_K);
        if (n_pieces * HEAD_TILE_M > 0x7FFFFFFFll) return fail(TFE_ERR_INVALID_ARG);      // TMA coordinates are 32-bit
        if (cudaMalloc(&h->d_w_tiled, (size_t)n_pieces * HEAD_TILE_M * 128) != cudaSuccess) return fail(TFE_ERR_CUDA);
        tfe_head_retile_kernel<<<h->sm_count * 8, 256>>>(static_cast<const uint4 *>(w_pref), static_cast<uint4 *>(h->d_w_tiled), V, d,
                                                        h->rows_per_cta, h->tiles_per_cta, n_pieces);
        if (cudaGetLastError() != cudaSuccess || cudaDeviceSynchronize() != cudaSuccess) return fail(TFE_ERR_CUDA);
        const uint64_t rows = (uint64_t)n_pieces * HEAD_TILE_M;
        if (!make_map(&h->map_w, h->d_w_tiled, rows, HEAD_TILE_K, HEAD_TILE_M)) return fail(TFE_ERR_CUDA);
        if (!make_map(&h->map_w_tail, h->d_w_tiled, rows, HEAD_TILE_K, h->tail_rows ? (uint32_t)h->tail_rows : 8u))
            return fail(TFE_ERR_CUDA);
    }
    h->n_fine = h->grid * h->tiles_per_cta * 4;
    if (h->n_fine > HEAD_MAX_FINE) return fail(TFE_ERR_INVALID_ARG);      // a vocabulary beyond 148 x 14 tiles of 128 rows
    const size_t nb = (size_t)max_batch;
    if (cudaMalloc(&h->d_logits, nb * (size_t)h->ld * sizeof(float)) != cudaSuccess) return fail(TFE_ERR_CUDA);
    if (cudaMalloc(&h->d_lse, nb * sizeof(float)) != cudaSuccess) return fail(TFE_ERR_CUDA);
    if (cudaMalloc(&h->d_status, sizeof(uint32_t)) != cudaSuccess) return fail(TFE_ERR_CUDA);
    if (cudaMemset(h->d_status, 0, sizeof(uint32_t)) != cudaSuccess) return fail(TFE_ERR_CUDA);
    if (cudaMalloc(&h->d_group_max, nb * 4 * (size_t)h->grid * sizeof(float)) != cudaSuccess) return fail(TFE_ERR_CUDA);
    if (cudaMalloc(&h->d_group_sum, nb * 4 * (size_t)h->grid * sizeof(float)) != cudaSuccess) return fail(TFE_ERR_CUDA);
    if (cudaMalloc(&h->d_fine_max, nb * (size_t)h->n_fine * sizeof(float)) != cudaSuccess) return fail(TFE_ERR_CUDA);
    if (cudaFuncSetAttribute(tfe_head_gemm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, HEAD_DYN_SMEM) !=
        cudaSuccess)
        return fail(TFE_ERR_CUDA);
    *out = h;
    return TFE_OK;
}

void tfe_head_destroy(tfe_head *h)
{
    if (!h) return;
    int prev = 0;
    (void)cudaGetDevice(&prev);
    (void)cudaSetDevice(h->device);
    (void)cudaDeviceSynchronize();
    if (h->d_w_tiled) (void)cudaFree(h->d_w_tiled);
    if (h->d_logits) (void)cudaFree(h->d_logits);
    if (h->d_lse) (void)cudaFree(h->d_lse);
    if (h->d_status) (void)cudaFree(h->d_status);
    if (h->d_group_max) (void)cudaFree(h->d_group_max);
    if (h->d_group_sum) (void)cudaFree(h->d_group_sum);
    if (h->d_fine_max) (void)cudaFree(h->d_fine_max);
    (void)cudaSetDevice(prev);
    delete h;
}

tfe_status tfe_head_topk(tfe_head *h, const void *hidden, int32_t B, int32_t K, int32_t *cand_tokens,
                         float *cand_prob, void *stream_)
{
    if (!h || B < 0 || B > h->max_batch || K < 1 || K > HEAD_MAX_K || K > h->V) return TFE_ERR_INVALID_ARG;
    if (B == 0) return TFE_OK;
    if (!hidden || !cand_tokens || !cand_prob) return TFE_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(hidden) & 15u) != 0) return TFE_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    HeadGemmParams g{};
    g.V = h->V; g.d = h->d; g.B = B;
    g.N = (B + 15) / 16 * 16;
    g.rows_per_cta = h->rows_per_cta; g.tail_rows = h->tail_rows;
    const uint32_t stage_bytes = HEAD_TILE_M * 128u + (uint32_t)g.N * 128u;
    const uint32_t budget = HEAD_DYN_SMEM - 1024;               // minus the alignment slack
    g.stages = (int32_t)std::min<uint32_t>(HEAD_MAX_STAGES, budget / stage_bytes);
    if (g.stages < 2) return TFE_ERR_INTERNAL;
    uint32_t cols = 32;
    while (cols < 2u * (uint32_t)g.N) cols <<= 1;
    g.tmem_cols = cols;
    g.logits = h->d_logits; g.ld = h->ld; g.status = h->d_status; g.group_max = h->d_group_max;
    g.group_sum = h->d_group_sum; g.fine_max = h->d_fine_max; g.n_fine = h->n_fine; g.tiles_per_cta = h->tiles_per_cta;
    CUtensorMap map_h;
    if (!make_map(&map_h, hidden, (uint64_t)B, (uint64_t)h->d, (uint32_t)g.N)) return TFE_ERR_CUDA;
    const size_t smem = (size_t)g.stages * stage_bytes + 1024;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)h->grid); cfg.blockDim = dim3(HEAD_THREADS); cfg.dynamicSmemBytes = smem; cfg.stream = stream;
    cfg.attrs = attr; cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, tfe_head_gemm_kernel, h->map_w, h->map_w_tail, map_h, g) != cudaSuccess) {
        (void)cudaGetLastError();
        return TFE_ERR_CUDA;
    }

    HeadSelParams s{};
    s.logits = h->d_logits; s.ld = h->ld; s.V = h->V; s.B = B; s.K = K;
    s.out_tokens = cand_tokens; s.out_prob = cand_prob; s.out_lse = h->d_lse;
    s.group_max = h->d_group_max; s.group_sum = h->d_group_sum; s.groups = 4 * h->grid;
    s.fine_max = h->d_fine_max; s.n_fine = h->n_fine; s.tiles_per_cta = h->tiles_per_cta; s.rows_per_cta = h->rows_per_cta;
    cfg.gridDim = dim3((unsigned)B); cfg.blockDim = dim3(HEAD_SEL_THREADS); cfg.dynamicSmemBytes = 0;
    if (cudaLaunchKernelEx(&cfg, tfe_head_select_kernel, s) != cudaSuccess) { (void)cudaGetLastError(); return TFE_ERR_CUDA; }
    return TFE_OK;
}

tfe_status tfe_head_buffers(tfe_head *h, const float **logits, int64_t *ld, const float **lse)
{
    if (!h) return TFE_ERR_INVALID_ARG;
    if (logits) *logits = h->d_logits;
    if (ld) *ld = h->ld;
    if (lse) *lse = h->d_lse;
    return TFE_OK;
}

tfe_status tfe_head_status(tfe_head *h, uint32_t *device_flags, void *stream_)
{
    if (!h || !device_flags) return TFE_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (cudaMemcpyAsync(device_flags, h->d_status, sizeof(uint32_t), cudaMemcpyDeviceToHost, stream) != cudaSuccess)
        return TFE_ERR_CUDA;
    if (cudaStreamSynchronize(stream) != cudaSuccess) return TFE_ERR_CUDA;
    return *device_flags ? TFE_ERR_INTERNAL : TFE_OK;
}

tfe_status tfe_head_geometry(const tfe_head *h, int32_t *grid, int32_t *rows_per_cta, int32_t *tail_rows)
{
    if (!h) return TFE_ERR_INVALID_ARG;
    if (grid) *grid = h->grid;
    if (rows_per_cta) *rows_per_cta = h->rows_per_cta;
    if (tail_rows) *tail_rows = h->tail_rows;
    return TFE_OK;
}

}  // extern "C"

#ifdef HEAD_TIMELINE
extern "C" int tfe_head_debug_timeline(long long *host16)
{
    return (int)cudaMemcpyFromSymbol(host16, g_head_tl, sizeof(long long) * 16);
}
#endif
