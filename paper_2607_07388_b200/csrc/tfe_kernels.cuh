// Device kernels of the Engram lookup-and-inject library (sm_100a).
//
//   tfe_insert_kernel          index build: place (key -> phrase id, residency) by atomicCAS
//   tfe_lookup_inject_kernel   the hot path: keys -> probe -> select -> tier -> gather -> inject
//                              -> order-stable miss compaction, one launch
//   tfe_install_kernel         write fetched rows into GPU-tier slots, update residency
//
// Index layout: an array of 128-byte buckets, 8 slots of {key64, val64} each.
// val64 = phrase id (high 32 bits) | residency (low 32 bits as int32: >= 0 GPU-tier
// slot, -1 host DRAM, -2 SSD).  Linear probing over buckets; keys are never
// removed, so a bucket with an empty slot ends the probe sequence of every key
// that would have passed through it.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "tfe_key.cuh"

#define TFE_BLOCK_THREADS 256
#define TFE_WARPS_PER_BLOCK (TFE_BLOCK_THREADS / 32)
#define TFE_NONE64 0xFFFFFFFFFFFFFFFFull
#define TFE_WAIT_LIMIT (8u << 20)      // polls of ~0.25 us each before a wait gives up

// device status bits (counters[TFE_CTR_STATUS])
#define TFE_DEV_WAIT_EXPIRED 1u
#define TFE_DEV_PROBE_LIMIT 2u
#define TFE_DEV_DUP_KEY 4u

struct TfeLookupParams {
    const int32_t *tokens;
    int32_t B, T, q_start, Tq;
    uint32_t Q;
    const ulonglong2 *index;
    uint64_t n_buckets;
    int32_t max_probe;
    const int4 *phrase_tokens;      // [N] token tuples, only read for hashed orders
    const uint4 *rows;              // GPU tier, [C][d] bf16
    int32_t d;
    const void *h;
    void *out;
    int32_t n_orders;
    int32_t orders[4];
    int32_t tok_bits;
    int32_t vocab;
    float lambda;
    uint32_t *sel_phrase;           // optional outputs
    int32_t *sel_slot;
    uint8_t *flags;
    uint32_t *scr_phrase;           // context scratch, [Q*cols]
    uint8_t *scr_flag;
    uint32_t *miss_q, *miss_phrase; // context miss list, [Q*cols]
    uint8_t *miss_tier;
    uint32_t *counters;             // TFE_CTR_* words
    unsigned long long *block_state;// [block_state_len] (epoch << 32) | misses of that block
    uint32_t block_state_len, q_per_block;
};

// Device-resident launch state (uint32 words).  A lookup launch numbers its blocks with TICKET,
// tags what it publishes with EPOCH, and its last block to finish resets TICKET / DONE, moves
// RUNNING to TOTAL and advances EPOCH.  EPOCH starts at 1; tag 0 means "never written".
enum { TFE_CTR_RUNNING = 0, TFE_CTR_TOTAL = 1, TFE_CTR_STATUS = 2, TFE_CTR_TICKET = 3, TFE_CTR_DONE = 4,
       TFE_CTR_EPOCH = 5, TFE_CTR_WORDS = 8 };

// ------------------------------------------------------------------ index build

__global__ void tfe_insert_kernel(ulonglong2 *index, uint64_t n_buckets, int max_probe,
                                  const uint64_t *keys, const int32_t *slot_state, uint32_t n,
                                  uint32_t *phrase_pos, uint32_t *status)
{
    uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const uint64_t key = keys[i];
    const uint64_t val = ((uint64_t)i << 32) | (uint32_t)slot_state[i];
    uint64_t bucket = tfe_home_bucket_of(key, n_buckets);
    for (int probe = 0; probe < max_probe; ++probe) {
        for (int s = 0; s < TFE_SLOTS_PER_BUCKET; ++s) {
            ulonglong2 *slot = index + bucket * TFE_SLOTS_PER_BUCKET + s;
            unsigned long long seen = *(volatile unsigned long long *)&slot->x;
            if (seen == 0ull) seen = atomicCAS(&slot->x, 0ull, (unsigned long long)key);
            if (seen == 0ull) {
                slot->y = val;
                phrase_pos[i] = (uint32_t)(bucket * TFE_SLOTS_PER_BUCKET + s);
                return;
            }
            if (seen == key) { atomicOr(status, TFE_DEV_DUP_KEY); return; }
        }
        bucket = bucket + 1 == n_buckets ? 0 : bucket + 1;
    }
    atomicOr(status, TFE_DEV_PROBE_LIMIT);
}

// -------------------------------------------------------------- small helpers

__device__ __forceinline__ uint4 ld_stream(const uint4 *p)   // touched once: do not keep in L1
{
    uint4 v;
    asm volatile("ld.global.cs.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
__device__ __forceinline__ void st_stream(uint4 *p, uint4 v)
{
    asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};"
                 :: "l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
__device__ __forceinline__ uint4 ld_row(const uint4 *p)      // read-only table data
{
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
__device__ __forceinline__ uint2 ld_row2(const uint2 *p)
{
    uint2 v;
    asm volatile("ld.global.nc.L1::no_allocate.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "l"(p));
    return v;
}
__device__ __forceinline__ ulonglong2 ld_slot(const ulonglong2 *p)
{
    ulonglong2 v;
    asm volatile("ld.global.nc.v2.u64 {%0,%1}, [%2];" : "=l"(v.x), "=l"(v.y) : "l"(p));
    return v;
}
__device__ __forceinline__ float bf_lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf_hi(uint32_t u) { return __uint_as_float(u & 0xFFFF0000u); }
__device__ __forceinline__ uint32_t pack_bf2(float lo, float hi)   // round to nearest even
{
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&v);
}
__device__ __forceinline__ float warp_sum(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    return v;
}

// Stored tuples are in stream order (st.x oldest); tk[j] is the token j places before the query.
__device__ __forceinline__ bool tuple_matches(const int4 st, const int32_t (&tk)[4], int n)
{
    switch (n) {
    case 1: return st.x == tk[0];
    case 2: return st.x == tk[1] && st.y == tk[0];
    case 3: return st.x == tk[2] && st.y == tk[1] && st.z == tk[0];
    default: return st.x == tk[3] && st.y == tk[2] && st.z == tk[1] && st.w == tk[0];
    }
}

// The retained GPU-resident rows of one query and their aggregation weights.
struct TfeRowSet {
    const uint4 *ptr[4];
    float alpha[4];
    int n;
};

// Elements handled by one lane in one step: 8 (bf16 hidden: one 16-byte vector of h,
// of the row and of out) or 4 (fp32 hidden: 16 bytes of h / out, 8 bytes of the row).
template <int HT> struct TfeVec;
template <> struct TfeVec<0> { static constexpr int N = 8; typedef uint4 RowRaw; };
template <> struct TfeVec<1> { static constexpr int N = 4; typedef uint2 RowRaw; };

template <int HT>
__device__ __forceinline__ void unpack_hidden(const uint4 raw, float (&x)[TfeVec<HT>::N])
{
    if constexpr (HT == 0) {
        x[0] = bf_lo(raw.x); x[1] = bf_hi(raw.x); x[2] = bf_lo(raw.y); x[3] = bf_hi(raw.y);
        x[4] = bf_lo(raw.z); x[5] = bf_hi(raw.z); x[6] = bf_lo(raw.w); x[7] = bf_hi(raw.w);
    } else {
        x[0] = __uint_as_float(raw.x); x[1] = __uint_as_float(raw.y);
        x[2] = __uint_as_float(raw.z); x[3] = __uint_as_float(raw.w);
    }
}

template <int HT>
__device__ __forceinline__ typename TfeVec<HT>::RowRaw ld_row_raw(const uint4 *row, int step_idx)
{
    if constexpr (HT == 0) return ld_row(row + step_idx);
    else return ld_row2(reinterpret_cast<const uint2 *>(row) + step_idx);
}

template <int HT>
__device__ __forceinline__ void unpack_row(const typename TfeVec<HT>::RowRaw r, float (&e)[TfeVec<HT>::N])
{
    e[0] = bf_lo(r.x); e[1] = bf_hi(r.x); e[2] = bf_lo(r.y); e[3] = bf_hi(r.y);
    if constexpr (HT == 0) {
        e[4] = bf_lo(r.z); e[5] = bf_hi(r.z); e[6] = bf_lo(r.w); e[7] = bf_hi(r.w);
    }
}

template <int HT>
__device__ __forceinline__ void load_hidden(const void *hrow, int step_idx, float (&x)[TfeVec<HT>::N])
{
    unpack_hidden<HT>(ld_stream(reinterpret_cast<const uint4 *>(hrow) + step_idx), x);
}

template <int HT>
__device__ __forceinline__ void load_row(const uint4 *row, int step_idx, float (&e)[TfeVec<HT>::N])
{
    unpack_row<HT>(ld_row_raw<HT>(row, step_idx), e);
}

template <int HT>
__device__ __forceinline__ void store_hidden(void *orow, int step_idx, const float (&y)[TfeVec<HT>::N])
{
    uint4 v;
    if constexpr (HT == 0) {
        v.x = pack_bf2(y[0], y[1]); v.y = pack_bf2(y[2], y[3]);
        v.z = pack_bf2(y[4], y[5]); v.w = pack_bf2(y[6], y[7]);
    } else {
        v.x = __float_as_uint(y[0]); v.y = __float_as_uint(y[1]);
        v.z = __float_as_uint(y[2]); v.w = __float_as_uint(y[3]);
    }
    st_stream(reinterpret_cast<uint4 *>(orow) + step_idx, v);
}

// m = sum_r alpha_r * row_r for this lane's elements of one step (fp32, ascending order).
template <int HT, bool ALL>
__device__ __forceinline__ void load_memory(const TfeRowSet &rs, int step_idx, float (&m)[TfeVec<HT>::N])
{
    if constexpr (!ALL) {
        load_row<HT>(rs.ptr[0], step_idx, m);
    } else {
#pragma unroll
        for (int k = 0; k < TfeVec<HT>::N; ++k) m[k] = 0.f;
        for (int r = 0; r < rs.n; ++r) {
            float e[TfeVec<HT>::N];
            load_row<HT>(rs.ptr[r], step_idx, e);
#pragma unroll
            for (int k = 0; k < TfeVec<HT>::N; ++k) m[k] = fmaf(rs.alpha[r], e[k], m[k]);
        }
    }
}

// --------------------------------------------------------------- the hot path
//
// Work split: block `rank` (ticket order) owns the contiguous query range
// [rank*q_per_block, ...); its warps take queries from that range one at a time
// through a shared counter.  One warp per query:
//   * four 8-lane groups, one per configured order, form their key and scan one
//     128-byte index bucket per load (one coalesced request per group);
//   * the warp picks the retained phrase(s), classifies the tier, records the
//     result, then streams h -> out for the row, adding g*m for GPU hits.
// Misses are compacted at the end of the block: blocks publish their miss count,
// a block that has misses adds up the counts of all lower-ranked blocks (they were
// started earlier and never wait on it) and writes its entries behind them, so the
// list comes out in ascending (q, order) without a second launch.
template <int HT, bool ALL, bool COS>
__global__ void __launch_bounds__(TFE_BLOCK_THREADS, (!ALL && !COS) ? 4 : 2)
tfe_lookup_inject_kernel(const TfeLookupParams p)
{
    constexpr int VN = TfeVec<HT>::N;
    constexpr int UNROLL = ALL ? 2 : 4;
    __shared__ uint32_t s_rank, s_epoch, s_next, s_any_miss;
    __shared__ uint32_t s_red[TFE_WARPS_PER_BLOCK];
    __shared__ uint32_t s_scan_base;

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int grp = lane >> 3, sub = lane & 7;
    if (threadIdx.x == 0) {
        s_rank = atomicAdd(&p.counters[TFE_CTR_TICKET], 1u);
        s_epoch = *(volatile uint32_t *)&p.counters[TFE_CTR_EPOCH];
        s_next = 0;
        s_any_miss = 0;
    }
    __syncthreads();
    const uint32_t rank = s_rank, epoch = s_epoch;
    const uint32_t q_begin = min(p.Q, rank * p.q_per_block);
    const uint32_t q_end = min(p.Q, q_begin + p.q_per_block);
    const int cols = ALL ? p.n_orders : 1;
    const int steps = p.d / VN;                  // 16-byte steps of h per row
    const size_t hid_row_bytes = (size_t)p.d * (HT == 0 ? 2 : 4);
    const bool in_place = p.out == p.h;

    const int my_order = grp < p.n_orders ? p.orders[grp] : 0;
    const bool my_hashed = my_order > 0 && !tfe_order_is_packed(my_order, p.tok_bits);

    for (;;) {
        uint32_t lq = 0;
        if (lane == 0) lq = atomicAdd(&s_next, 1u);
        lq = __shfl_sync(0xFFFFFFFFu, lq, 0);
        if (lq >= q_end - q_begin) break;
        const uint32_t q = q_begin + lq;
        const uint32_t b = q / (uint32_t)p.Tq;
        const int32_t t = p.q_start + (int32_t)(q - b * (uint32_t)p.Tq);

        // ---- trailing n-gram keys: lane `sub` of every group fetches the token at t - sub
        int32_t tk_mine = -1;
        if (sub < 4 && t - sub >= 0) {
            tk_mine = __ldg(p.tokens + (size_t)b * p.T + (t - sub));
            if ((uint32_t)tk_mine >= (uint32_t)p.vocab) tk_mine = -1;
        }
        int32_t tk[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) tk[j] = __shfl_sync(0xFFFFFFFFu, tk_mine, (lane & ~7) + j);
        bool active = my_order > 0;
#pragma unroll
        for (int j = 0; j < 4; ++j)
            if (j < my_order && tk[j] < 0) active = false;
        const uint64_t key = active ? tfe_make_key(my_order, tk, p.tok_bits) : 0ull;

        // ---- exact-match probe: 8 lanes scan one bucket per iteration
        uint64_t bucket = active ? tfe_home_bucket_of(key, p.n_buckets) : 0ull;
        unsigned long long found = TFE_NONE64;
        for (int probe = 0; probe < p.max_probe; ++probe) {
            if (!__any_sync(0xFFFFFFFFu, active)) break;
            ulonglong2 s = make_ulonglong2(0ull, 0ull);
            if (active) s = ld_slot(p.index + bucket * TFE_SLOTS_PER_BUCKET + sub);
            const uint32_t hit = __ballot_sync(0xFFFFFFFFu, active && s.x == key);
            const uint32_t emp = __ballot_sync(0xFFFFFFFFu, active && s.x == 0ull);
            const uint32_t ghit = (hit >> (grp * 8)) & 0xFFu, gemp = (emp >> (grp * 8)) & 0xFFu;
            const int src = (lane & ~7) + (ghit ? __ffs(ghit) - 1 : 0);
            const unsigned long long v = __shfl_sync(0xFFFFFFFFu, s.y, src);
            if (active) {
                if (ghit) { found = v; active = false; }
                else if (gemp) active = false;
                else bucket = bucket + 1 == p.n_buckets ? 0 : bucket + 1;
            }
        }
        // hashed orders: a key match is confirmed against the stored token tuple
        if (my_hashed && found != TFE_NONE64) {
            const int4 st = __ldg(p.phrase_tokens + (uint32_t)(found >> 32));
            if (!tuple_matches(st, tk, my_order)) found = TFE_NONE64;
        }

        // ---- selection policy + tier walk (all lanes hold all four group results)
        unsigned long long res[4];
#pragma unroll
        for (int g = 0; g < 4; ++g) res[g] = __shfl_sync(0xFFFFFFFFu, found, g * 8);

        TfeRowSet rs;
        rs.n = 0;
        if (!ALL) {
            unsigned long long sel = TFE_NONE64;
#pragma unroll
            for (int g = 0; g < 4; ++g)
                if (g < p.n_orders && res[g] != TFE_NONE64) sel = res[g];
            uint32_t phrase = TFE_NONE64 & 0xFFFFFFFFu;
            int32_t slot = -3;
            uint8_t flag = 0;
            if (sel != TFE_NONE64) {
                phrase = (uint32_t)(sel >> 32);
                slot = (int32_t)(uint32_t)sel;
                flag = slot >= 0 ? 1 : (slot == -1 ? 2 : 3);
                if (slot < -2) slot = -2;
            }
            if (lane == 0) {
                p.scr_flag[q] = flag;
                p.scr_phrase[q] = phrase;
                if (p.flags) p.flags[q] = flag;
                if (p.sel_phrase) p.sel_phrase[q] = phrase;
                if (p.sel_slot) p.sel_slot[q] = slot;
                if (flag >= 2) s_any_miss = 1;
            }
            if (flag == 1) {
                rs.n = 1;
                rs.ptr[0] = p.rows + (size_t)slot * (size_t)(p.d / 8);
                rs.alpha[0] = 1.f;
            }
        } else {
            int n_sum = 0;
#pragma unroll
            for (int g = 0; g < 4; ++g)
                if (g < p.n_orders && res[g] != TFE_NONE64) n_sum += p.orders[g];
#pragma unroll
            for (int g = 0; g < 4; ++g) {
                if (g >= p.n_orders) continue;
                uint32_t phrase = TFE_NONE64 & 0xFFFFFFFFu;
                int32_t slot = -3;
                uint8_t flag = 0;
                if (res[g] != TFE_NONE64) {
                    phrase = (uint32_t)(res[g] >> 32);
                    slot = (int32_t)(uint32_t)res[g];
                    flag = slot >= 0 ? 1 : (slot == -1 ? 2 : 3);
                    if (slot < -2) slot = -2;
                }
                if (lane == g) {
                    const size_t k = (size_t)q * cols + g;
                    p.scr_flag[k] = flag;
                    p.scr_phrase[k] = phrase;
                    if (p.flags) p.flags[k] = flag;
                    if (p.sel_phrase) p.sel_phrase[k] = phrase;
                    if (p.sel_slot) p.sel_slot[k] = slot;
                    if (flag >= 2) s_any_miss = 1;
                }
                if (flag == 1) {
                    rs.ptr[rs.n] = p.rows + (size_t)slot * (size_t)(p.d / 8);
                    rs.alpha[rs.n] = (float)p.orders[g] / (float)n_sum;
                    ++rs.n;
                }
            }
        }

        // ---- gather + gated residual injection: out = h + g * m
        const char *hrow = reinterpret_cast<const char *>(p.h) + (size_t)q * hid_row_bytes;
        char *orow = reinterpret_cast<char *>(p.out) + (size_t)q * hid_row_bytes;
        if (rs.n == 0) {
            if (!in_place) {
                for (int s0 = 0; s0 < steps; s0 += 32 * 4) {
                    uint4 v[4];
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const int i = s0 + u * 32 + lane;
                        if (i < steps) v[u] = ld_stream(reinterpret_cast<const uint4 *>(hrow) + i);
                    }
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const int i = s0 + u * 32 + lane;
                        if (i < steps) st_stream(reinterpret_cast<uint4 *>(orow) + i, v[u]);
                    }
                }
            }
            continue;
        }
        float gate = p.lambda;
        if (COS) {
            float sa = 0.f, sb = 0.f, sc = 0.f;      // <h,m>, <h,h>, <m,m>
            for (int i = lane; i < steps; i += 32) {
                float x[VN], m[VN];
                load_hidden<HT>(hrow, i, x);
                load_memory<HT, ALL>(rs, i, m);
#pragma unroll
                for (int k = 0; k < VN; ++k) {
                    sa = fmaf(x[k], m[k], sa); sb = fmaf(x[k], x[k], sb); sc = fmaf(m[k], m[k], sc);
                }
            }
            sa = warp_sum(sa); sb = warp_sum(sb); sc = warp_sum(sc);
            gate = p.lambda / (1.f + __expf(-sa * rsqrtf(fmaf(sb, sc, 1e-12f))));
        }
        if constexpr (!ALL) {
            // one row: keep the raw 16-byte vectors in flight, unpack when they are consumed
            for (int s0 = 0; s0 < steps; s0 += 32 * UNROLL) {
                uint4 hv[UNROLL];
                typename TfeVec<HT>::RowRaw rv[UNROLL];
#pragma unroll
                for (int u = 0; u < UNROLL; ++u) {
                    const int i = s0 + u * 32 + lane;
                    if (i < steps) {
                        hv[u] = ld_stream(reinterpret_cast<const uint4 *>(hrow) + i);
                        rv[u] = ld_row_raw<HT>(rs.ptr[0], i);
                    }
                }
#pragma unroll
                for (int u = 0; u < UNROLL; ++u) {
                    const int i = s0 + u * 32 + lane;
                    if (i < steps) {
                        float x[VN], m[VN], y[VN];
                        unpack_hidden<HT>(hv[u], x);
                        unpack_row<HT>(rv[u], m);
#pragma unroll
                        for (int k = 0; k < VN; ++k) y[k] = fmaf(gate, m[k], x[k]);
                        store_hidden<HT>(orow, i, y);
                    }
                }
            }
        } else {
            for (int s0 = 0; s0 < steps; s0 += 32 * UNROLL) {
                float x[UNROLL][VN], m[UNROLL][VN];
#pragma unroll
                for (int u = 0; u < UNROLL; ++u) {
                    const int i = s0 + u * 32 + lane;
                    if (i < steps) {
                        load_hidden<HT>(hrow, i, x[u]);
                        load_memory<HT, ALL>(rs, i, m[u]);
                    }
                }
#pragma unroll
                for (int u = 0; u < UNROLL; ++u) {
                    const int i = s0 + u * 32 + lane;
                    if (i < steps) {
                        float y[VN];
#pragma unroll
                        for (int k = 0; k < VN; ++k) y[k] = fmaf(gate, m[u][k], x[u][k]);
                        store_hidden<HT>(orow, i, y);
                    }
                }
            }
        }
    }

    // ---- order-stable miss compaction for this block's query range
    __syncthreads();
    const uint32_t n_ent = (q_end - q_begin) * (uint32_t)cols;
    const size_t ent0 = (size_t)q_begin * cols;
    uint32_t cnt = 0;
    if (s_any_miss) {
        for (uint32_t i = threadIdx.x; i < n_ent; i += TFE_BLOCK_THREADS) cnt += p.scr_flag[ent0 + i] >= 2;
        cnt = __reduce_add_sync(0xFFFFFFFFu, cnt);
        if (lane == 0) s_red[warp] = cnt;
        __syncthreads();
        cnt = 0;
#pragma unroll
        for (int w = 0; w < TFE_WARPS_PER_BLOCK; ++w) cnt += s_red[w];
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        if (cnt) atomicAdd(&p.counters[TFE_CTR_RUNNING], cnt);
        __threadfence();
        atomicExch(&p.block_state[rank], ((unsigned long long)epoch << 32) | cnt);
    }
    if (cnt != 0) {     // block-uniform
        // misses of all lower-ranked blocks (bounded wait; they publish when they finish)
        uint32_t before = 0;
        bool expired = false;
        for (uint32_t j = threadIdx.x; j < rank; j += TFE_BLOCK_THREADS) {
            unsigned long long v = 0;
            uint32_t polls = 0;
            for (;;) {
                v = *(volatile unsigned long long *)&p.block_state[j];
                if ((uint32_t)(v >> 32) == epoch) break;
                if (++polls > TFE_WAIT_LIMIT) { expired = true; break; }
                __nanosleep(200);
            }
            if (!expired) before += (uint32_t)v;
        }
        const int any_expired = __syncthreads_or(expired);
        before = __reduce_add_sync(0xFFFFFFFFu, before);
        if (lane == 0) s_red[warp] = before;
        __syncthreads();
        if (threadIdx.x == 0) {
            uint32_t tot = 0;
            for (int w = 0; w < TFE_WARPS_PER_BLOCK; ++w) tot += s_red[w];
            s_scan_base = tot;
            if (any_expired) atomicOr(&p.counters[TFE_CTR_STATUS], TFE_DEV_WAIT_EXPIRED);
        }
        __syncthreads();
        if (!any_expired) {
            for (uint32_t i0 = 0; i0 < n_ent; i0 += TFE_BLOCK_THREADS) {
                const uint32_t i = i0 + threadIdx.x;
                uint8_t flag = 0;
                if (i < n_ent) flag = p.scr_flag[ent0 + i];
                const bool is_miss = flag >= 2;
                const uint32_t bal = __ballot_sync(0xFFFFFFFFu, is_miss);
                if (lane == 0) s_red[warp] = __popc(bal);
                __syncthreads();
                uint32_t off = s_scan_base;
                for (int w = 0; w < warp; ++w) off += s_red[w];
                off += __popc(bal & ((1u << lane) - 1u));
                if (is_miss) {
                    p.miss_q[off] = q_begin + i / (uint32_t)cols;
                    p.miss_phrase[off] = p.scr_phrase[ent0 + i];
                    p.miss_tier[off] = flag;
                }
                __syncthreads();
                if (threadIdx.x == 0) {
                    uint32_t tot = 0;
                    for (int w = 0; w < TFE_WARPS_PER_BLOCK; ++w) tot += s_red[w];
                    s_scan_base += tot;
                }
                __syncthreads();
            }
        }
    }

    // ---- the block that finishes last closes the call: it publishes the miss total and re-arms
    // the ticket / done counters and the epoch for the next launch (all state lives on the device,
    // so a launch can be replayed with unchanged parameters)
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        if (atomicAdd(&p.counters[TFE_CTR_DONE], 1u) == gridDim.x - 1) {
            __threadfence();
            p.counters[TFE_CTR_TOTAL] = atomicExch(&p.counters[TFE_CTR_RUNNING], 0u);
            p.counters[TFE_CTR_TICKET] = 0;
            p.counters[TFE_CTR_DONE] = 0;
            uint32_t next = epoch + 1;
            if (next == 0) {      // the tag wrapped: forget every stale tag before reusing values
                for (uint32_t j = 0; j < p.block_state_len; ++j) p.block_state[j] = 0ull;
                next = 1;
            }
            p.counters[TFE_CTR_EPOCH] = next;
        }
    }
}

// ------------------------------------------------------------- cache install

// One warp per installed row: the previous owner of the slot falls back to the
// host tier, the row is copied in, the phrase's index value becomes {id, slot}.
__global__ void __launch_bounds__(TFE_BLOCK_THREADS)
tfe_install_kernel(ulonglong2 *index, const uint32_t *phrase_pos, uint32_t *slot_owner, uint4 *rows,
                   int32_t row_vecs, int32_t n, const uint32_t *ids, const uint4 *src,
                   const int32_t *dst_slots)
{
    const int lane = threadIdx.x & 31;
    const int k = blockIdx.x * TFE_WARPS_PER_BLOCK + (threadIdx.x >> 5);
    if (k >= n) return;
    const uint32_t id = ids[k];
    const int32_t dst = dst_slots[k];
    if (lane == 0) {
        const uint32_t prev = slot_owner[dst];
        if (prev != 0xFFFFFFFFu)
            index[phrase_pos[prev]].y = ((unsigned long long)prev << 32) | 0xFFFFFFFFull;   // -1: host tier
        index[phrase_pos[id]].y = ((unsigned long long)id << 32) | (uint32_t)dst;
        slot_owner[dst] = id;
    }
    const uint4 *s = src + (size_t)k * row_vecs;
    uint4 *o = rows + (size_t)dst * row_vecs;
    for (int i = lane; i < row_vecs; i += 32) o[i] = ld_stream(s + i);
}
