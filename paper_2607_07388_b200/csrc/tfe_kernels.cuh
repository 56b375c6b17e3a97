// Device kernels of the Engram lookup-and-inject library (sm_100a).
//
//   tfe_lookup_inject_kernel   the hot path: keys -> probe -> select -> tier -> gather -> inject
//                              -> order-stable miss compaction, one launch
//   tfe_install_kernel         write fetched rows into GPU-tier slots, update residency
//
// Index layout: an array of 64-byte buckets, 4 slots of {key64, val64} each, filled by
// two-choice cuckoo hashing on the host: a key lives in one of its two buckets, so a
// lookup is exactly two independent 64-byte reads and never a dependent chain.
// val64 = phrase id (high 32 bits) | residency (low 32 bits as int32: >= 0 GPU-tier
// slot, -1 host DRAM, -2 SSD).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "tfe_key.cuh"

#ifndef TFE_BLOCK_THREADS
#define TFE_BLOCK_THREADS 256     // 8 warps; 3 blocks per SM within 80 registers per thread measured best
#endif
#define TFE_WARPS_PER_BLOCK (TFE_BLOCK_THREADS / 32)
#define TFE_NONE64 0xFFFFFFFFFFFFFFFFull

// device status bits (counters[TFE_CTR_STATUS])
#define TFE_DEV_PROBE_LIMIT 2u
#define TFE_DEV_DUP_KEY 4u
#define TFE_DEV_RECORD_TIMEOUT 8u      // the block that closes a call gave up waiting for a block's report or a record

// Division by a divisor fixed per call: q = (n * mul) >> shr, exact for every n < 2^31
// (mul = floor(2^shr / d) + 1, shr = 31 + ceil(log2 d); the host computes both).
struct TfeFastDiv { uint32_t mul, shr; };

// Programmatic dependent launch: a lookup launched with the stream-serialisation attribute may be set up
// while the kernel before it on the stream is still draining; it must not touch global memory before
// this point, where it waits until that kernel has completed and its writes are visible.  No early
// trigger is issued for the kernel after it (measured: successors that become resident early and sit
// waiting cost more than the hidden launch latency gains).  Without the attribute this is a no-op.
__device__ __forceinline__ void tfe_grid_dependency_sync()
{
    asm volatile("griddepcontrol.wait;" ::: "memory");
}

struct TfeLookupParams {
    const int32_t *tokens;
    int32_t B, T, q_start, Tq;
    uint32_t Q;
    TfeFastDiv div_tq;              // division by Tq
    uint32_t qb;                    // queries per warp batch, 1..8
    uint32_t q_lo, q_hi;            // LONGEST / CONST kernel: this launch handles queries [q_lo, q_hi) of the call
    uint32_t finalize;              // 1: this launch closes the call (builds the miss list over all Q queries)
    const ulonglong2 *index;
    uint64_t n_buckets;
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
    uint32_t lambda_bf16x2;         // lambda twice as bf16, valid when it is exactly a bf16 number
    uint32_t *sel_phrase;           // optional outputs
    int32_t *sel_slot;
    uint8_t *flags;
    unsigned long long *scr_rec;    // context scratch, [Q*cols] result records (tfe_make_record)
    uint32_t *miss_q, *miss_phrase; // context miss list, [Q*cols]
    uint8_t *miss_tier;
    uint32_t *counters;             // TFE_CTR_* words
    uint2 *slot_stats;              // per GPU-tier slot {injections since install, epoch of the last one}, or nullptr
    uint32_t *epoch;                // lookups completed so far (device word), with slot_stats
};

// Device-resident launch state (uint32 words; DONE and RUNNING form one 8-byte word that a single
// atomic updates).  Blocks of a lookup add their miss counts to RUNNING and tick DONE when they finish; the block that finishes last compacts the miss list,
// moves RUNNING to TOTAL and zeroes RUNNING / DONE for the next launch.  Because nothing of this
// lives in kernel parameters, a launch can be replayed unchanged.
// SEQ numbers the calls that have been closed on these counters: a call's records carry SEQ + 1 (its "tag"),
// which is how the block that builds the miss list tells a record of this call from what an earlier call left
// in the same place.
enum { TFE_CTR_DONE = 0, TFE_CTR_RUNNING = 1, TFE_CTR_TOTAL = 2, TFE_CTR_STATUS = 3, TFE_CTR_SEQ = 4, TFE_CTR_WORDS = 8 };

// One result record per (query, order column): tag (30 bits) | flag (2 bits) | phrase id (32 bits), written with
// a single 8-byte store, so whoever reads it sees all of it or an older record.
#define TFE_TAG_MASK 0x3FFFFFFFu
__device__ __forceinline__ uint32_t tfe_call_tag(const uint32_t *counters)
{
    const uint32_t tag = (__ldcg(counters + TFE_CTR_SEQ) + 1u) & TFE_TAG_MASK;
    return tag ? tag : 1u;           // 0 is what fresh (zeroed) scratch memory holds: never a call's tag
}
__device__ __forceinline__ unsigned long long tfe_make_record(uint32_t tag, uint32_t flag, uint32_t phrase)
{
    return ((unsigned long long)((tag << 2) | flag) << 32) | phrase;
}
#define TFE_SPIN_LIMIT (1u << 22)

// -------------------------------------------------------------- small helpers

__device__ __forceinline__ uint4 ld_stream(const uint4 *p)   // touched once: cached in L2 only
{
    uint4 v;
    asm volatile("ld.global.cg.v4.u32 {%0,%1,%2,%3}, [%4];"
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
__device__ __forceinline__ float bf_lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf_hi(uint32_t u) { return __uint_as_float(u & 0xFFFF0000u); }
__device__ __forceinline__ uint32_t pack_bf2(float lo, float hi)   // round to nearest even
{
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&v);
}
__device__ __forceinline__ uint32_t fma_bf16x2(uint32_t a, uint32_t b, uint32_t c)   // a*b + c per half
{
    uint32_t d;
    asm("fma.rn.bf16x2 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
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

// The index is what every call probes again; its lines ask to stay in L2 (evict-last), the hidden states that
// stream through ask to leave first (ld.global.cs / st.global.cs above).
__device__ __forceinline__ ulonglong4 ld_bucket32(const ulonglong4 *p)    // 32 bytes = two index slots
{
    ulonglong4 v;
    unsigned long long policy;
    asm("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(policy));
    asm volatile("ld.global.nc.L2::cache_hint.v4.u64 {%0,%1,%2,%3}, [%4], %5;"
                 : "=l"(v.x), "=l"(v.y), "=l"(v.z), "=l"(v.w) : "l"(p), "l"(policy));
    return v;
}

__device__ __forceinline__ uint32_t tfe_div(uint32_t n, TfeFastDiv d)
{
    return (uint32_t)(((unsigned long long)n * d.mul) >> d.shr);
}

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

// m = sum_r alpha_r * row_r for this lane's elements of one step (fp32, ascending order);
// LONGEST keeps one row with weight 1, which this reproduces exactly.
template <int HT, bool ALL>
__device__ __forceinline__ void load_memory(const uint4 *const (&rowp)[ALL ? 4 : 1], const float (&alpha)[ALL ? 4 : 1],
                                            int step_idx, float (&m)[TfeVec<HT>::N])
{
    if constexpr (!ALL) {
        load_row<HT>(rowp[0], step_idx, m);
    } else {
#pragma unroll
        for (int k = 0; k < TfeVec<HT>::N; ++k) m[k] = 0.f;
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            if (rowp[r] == nullptr) continue;
            float e[TfeVec<HT>::N];
            load_row<HT>(rowp[r], step_idx, e);
#pragma unroll
            for (int k = 0; k < TfeVec<HT>::N; ++k) m[k] = fmaf(alpha[r], e[k], m[k]);
        }
    }
}

// The ordered miss list of a call, built by one whole block: ascending entry index = ascending (q, order).
// `total` is the number of misses the blocks reported.  Every record is checked for this call's tag and read
// again (bounded) while it still shows an older one: the lookup kernels report without a fence, so a
// report can be seen before the records it covers.  The block then publishes TOTAL, closes the call (SEQ) and
// re-arms the launch state.
__device__ __forceinline__ void tfe_compact_misses(const TfeLookupParams &p, uint32_t total, int cols, uint32_t tag)
{
    __shared__ uint32_t s_scan;
    __shared__ uint32_t s_warp[32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int n_warps_blk = (blockDim.x + 31) >> 5;
    if (threadIdx.x == 0) s_scan = 0;
    __syncthreads();
    if (total != 0) {
        // order-stable compaction: every thread takes 4 consecutive records per round
        const uint32_t n_ent = p.Q * (uint32_t)cols;
        const uint32_t per_round = blockDim.x * 4;
        for (uint32_t e0 = 0; e0 < n_ent; e0 += per_round) {
            const uint32_t mine = e0 + threadIdx.x * 4;
            unsigned long long rec[4] = {0, 0, 0, 0};
            uint32_t cnt = 0;
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                if (mine + k >= n_ent) continue;
                const unsigned long long *src = p.scr_rec + mine + k;
                rec[k] = __ldcg(src);
                for (uint32_t spin = 0; (uint32_t)(rec[k] >> 34) != tag && spin < TFE_SPIN_LIMIT; ++spin) rec[k] = __ldcg(src);
                if ((uint32_t)(rec[k] >> 34) != tag) { atomicOr(&p.counters[TFE_CTR_STATUS], TFE_DEV_RECORD_TIMEOUT); rec[k] = 0; }
                cnt += (uint32_t)(rec[k] >> 33) & 1u;            // flags 2 and 3 have bit 1 set
            }
            uint32_t incl = cnt;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const uint32_t n = __shfl_up_sync(0xFFFFFFFFu, incl, o);
                if (lane >= o) incl += n;
            }
            if (lane == 31) s_warp[warp] = incl;
            __syncthreads();
            uint32_t off = s_scan + incl - cnt;
            for (int k = 0; k < warp; ++k) off += s_warp[k];
            if (cnt) {
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const uint32_t flag = (uint32_t)(rec[k] >> 32) & 3u;
                    if (flag >= 2) {
                        p.miss_q[off] = (mine + k) / (uint32_t)cols;
                        p.miss_phrase[off] = (uint32_t)rec[k];
                        p.miss_tier[off] = (uint8_t)flag;
                        ++off;
                    }
                }
            }
            __syncthreads();
            if (threadIdx.x == 0) {
                uint32_t t = 0;
                for (int k = 0; k < n_warps_blk; ++k) t += s_warp[k];
                s_scan += t;
            }
            __syncthreads();
        }
    }
    if (threadIdx.x == 0) {
        p.counters[TFE_CTR_TOTAL] = total;
        p.counters[TFE_CTR_DONE] = 0;
        p.counters[TFE_CTR_RUNNING] = 0;
        p.counters[TFE_CTR_SEQ] = tag;
        if (p.slot_stats != nullptr) *p.epoch = *p.epoch + 1;     // every block has read it by now
    }
}

// The hand-over from the blocks of a lookup to the one that builds the miss list is kept off the end of the
// launch, where a fence and an atomic round trip in every block would sit between the last byte of one launch
// and the first of the next (a decode call of 64 positions: 7.1 -> 5.1 us).  What the miss list needs is
// complete once a warp's last probe is on record, well before its last row has streamed, so:
//   * every WARP reports then (tfe_warp_probing_done): a shared-memory atomic, and from the warp that completes
//     its block one reduction on DONE / RUNNING that nobody waits for.  No fence: records carry the call's tag
//     and the reader checks it;
//   * the launch's last block (tfe_closing_block_epilogue, after its own rows) waits until DONE shows every
//     block -- all of them reported microseconds ago, unless the launch is tiny -- and builds the list.
// Every other block leaves with its last store.  The wait is bounded; the blocks of a launch are resident
// together (the grid never exceeds what the device holds), and a closing block that gives up says so in STATUS.
struct TfeProbeTick { unsigned long long warps_and_misses; };      // low word: warps reported, high word: their misses

__device__ __forceinline__ void tfe_warp_probing_done(const TfeLookupParams &p, TfeProbeTick *tick, uint32_t warp_miss)
{
    if ((threadIdx.x & 31) != 0) return;
    const uint32_t n_warps_blk = (blockDim.x + 31) >> 5;
    const unsigned long long before = atomicAdd(&tick->warps_and_misses, ((unsigned long long)warp_miss << 32) | 1ull);
    if ((uint32_t)before != n_warps_blk - 1) return;
    const unsigned long long block_miss = (before >> 32) + warp_miss;
    unsigned long long *dst = reinterpret_cast<unsigned long long *>(&p.counters[TFE_CTR_DONE]);
    asm volatile("red.global.add.u64 [%0], %1;" :: "l"(dst), "l"((block_miss << 32) | 1ull) : "memory");
}

__device__ __forceinline__ void tfe_closing_block_epilogue(const TfeLookupParams &p, int cols, uint32_t tag, bool finalize)
{
    if (blockIdx.x != gridDim.x - 1) return;
    __shared__ uint32_t s_total;
    if (threadIdx.x == 0) {                      // as soon as the first warp is through: the wait overlaps the other warps' rows
        const volatile unsigned long long *src = reinterpret_cast<const volatile unsigned long long *>(&p.counters[TFE_CTR_DONE]);
        unsigned long long v = *src;
        for (uint32_t spin = 0; (uint32_t)v != gridDim.x && spin < TFE_SPIN_LIMIT; ++spin) v = *src;
        if ((uint32_t)v != gridDim.x) atomicOr(&p.counters[TFE_CTR_STATUS], TFE_DEV_RECORD_TIMEOUT);
        s_total = (uint32_t)(v >> 32);
        if (!finalize) p.counters[TFE_CTR_DONE] = 0;      // a partial launch of a call issued in pieces: misses keep accumulating
    }
    __syncthreads();
    if (finalize) tfe_compact_misses(p, s_total, cols, tag);
}

// A GPU-tier slot served an injection in the lookup of epoch `epoch`.
__device__ __forceinline__ void tfe_touch_slot(uint2 *slot_stats, int32_t slot, uint32_t epoch)
{
    atomicAdd(&slot_stats[slot].x, 1u);
    slot_stats[slot].y = epoch;
}

// One lane's probe: the trailing n-gram of query q (n = this lane's order) -> key -> index value
// {phrase id, residency}, or TFE_NONE64 (no such phrase, n-gram reaches before the sequence
// start, or it holds an id outside [0, vocab)).  Three dependent steps: the token ids, both
// candidate buckets (4 x 32 bytes, all in flight together), and -- hashed orders only -- the
// stored tuple of a key match.
__device__ __forceinline__ unsigned long long tfe_probe_lane(const TfeLookupParams &p, uint32_t q, bool mine,
                                                             int my_order, bool my_hashed)
{
    unsigned long long found = TFE_NONE64;
    if (mine && my_order > 0) {
        const uint32_t b = tfe_div(q, p.div_tq);
        const int32_t t = p.q_start + (int32_t)(q - b * (uint32_t)p.Tq);
        int32_t tk[4] = {-1, -1, -1, -1};
        bool ok = t - (my_order - 1) >= 0;
        if (ok) {
            const int32_t *tp = p.tokens + (size_t)b * p.T + t;
#pragma unroll
            for (int j = 0; j < 4; ++j)
                if (j < my_order) {
                    tk[j] = __ldg(tp - j);
                    if ((uint32_t)tk[j] >= (uint32_t)p.vocab) ok = false;
                }
        }
        if (ok) {
            const uint64_t key = tfe_make_key(my_order, tk, p.tok_bits);
            const uint64_t b1 = tfe_home_bucket_of(key, p.n_buckets);
            const uint64_t b2 = tfe_second_bucket_of(key, b1, p.n_buckets);
            const ulonglong4 *p1 = reinterpret_cast<const ulonglong4 *>(p.index + b1 * TFE_SLOTS_PER_BUCKET);
            const ulonglong4 *p2 = reinterpret_cast<const ulonglong4 *>(p.index + b2 * TFE_SLOTS_PER_BUCKET);
            ulonglong4 w[4];                     // 2 buckets x 4 slots of {key, value}, all four loads in flight
            w[0] = ld_bucket32(p1); w[1] = ld_bucket32(p1 + 1);
            w[2] = ld_bucket32(p2); w[3] = ld_bucket32(p2 + 1);
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                if (w[k].x == key) found = w[k].y;
                if (w[k].z == key) found = w[k].w;
            }
            // hashed orders: a key match is confirmed against the stored token tuple
            if (my_hashed && found != TFE_NONE64) {
                const int4 st = __ldg(p.phrase_tokens + (uint32_t)(found >> 32));
                if (!tuple_matches(st, tk, my_order)) found = TFE_NONE64;
            }
        }
    }
    return found;
}

// LONGEST policy for the quad of lanes that probed one query: the match of greatest order is
// retained, its tier decides hit / miss, lane 4*ql records the result.  Returns (on that lane) the
// GPU-tier slot to add, or -1.
__device__ __forceinline__ int32_t tfe_select_longest(const TfeLookupParams &p, unsigned long long found, uint32_t q,
                                                      bool mine, int lane, uint32_t &my_miss, uint32_t tag)
{
    const uint32_t quad_found = (__ballot_sync(0xFFFFFFFFu, found != TFE_NONE64) >> (lane & ~3)) & 0xFu;
    const int top = quad_found ? 31 - __clz(quad_found) : 0;                   // greatest order that matched
    const unsigned long long sel = __shfl_sync(0xFFFFFFFFu, found, (lane & ~3) + top);
    int32_t my_slot = -1;
    if ((lane & 3) == 0 && mine) {
        uint32_t phrase = 0xFFFFFFFFu;
        int32_t st_ = -3;
        uint32_t flag = 0;
        if (quad_found) {
            phrase = (uint32_t)(sel >> 32);
            st_ = (int32_t)(uint32_t)sel;
            flag = st_ >= 0 ? 1 : (st_ == -1 ? 2 : 3);
        }
        if (flag == 1) my_slot = st_;
        p.scr_rec[q] = tfe_make_record(tag, flag, phrase);
        if (flag >= 2) ++my_miss;
        if (p.flags) p.flags[q] = (uint8_t)flag;
        if (p.sel_phrase) p.sel_phrase[q] = phrase;
        if (p.sel_slot) p.sel_slot[q] = st_;
    }
    return my_slot;
}

// The same for a query probed by the lanes base .. base + popc(group_mask) - 1 (two per order: both lanes of a
// pair hold the pair's result); the query's first lane records.
__device__ __forceinline__ int32_t tfe_select_longest_group(const TfeLookupParams &p, unsigned long long found, uint32_t q,
                                                            bool mine, int base, uint32_t group_mask, bool first_lane,
                                                            uint32_t &my_miss, uint32_t tag)
{
    const uint32_t group_found = (__ballot_sync(0xFFFFFFFFu, found != TFE_NONE64) >> base) & group_mask;
    const int top = group_found ? 31 - __clz(group_found) : 0;                 // a lane of the greatest order that matched
    const unsigned long long sel = __shfl_sync(0xFFFFFFFFu, found, base + top);
    int32_t my_slot = -1;
    if (first_lane && mine) {
        uint32_t phrase = 0xFFFFFFFFu;
        int32_t st_ = -3;
        uint32_t flag = 0;
        if (group_found) {
            phrase = (uint32_t)(sel >> 32);
            st_ = (int32_t)(uint32_t)sel;
            flag = st_ >= 0 ? 1 : (st_ == -1 ? 2 : 3);
        }
        if (flag == 1) my_slot = st_;
        p.scr_rec[q] = tfe_make_record(tag, flag, phrase);
        if (flag >= 2) ++my_miss;
        if (p.flags) p.flags[q] = (uint8_t)flag;
        if (p.sel_phrase) p.sel_phrase[q] = phrase;
        if (p.sel_slot) p.sel_slot[q] = st_;
    }
    return my_slot;
}

// --------------------------------------------------------------- the hot path
//
// One launch does everything, and every warp works on its own: it takes batches of `qb`
// queries (1..8; query lq of batch b is b + lq * n_batches, so neighbouring positions go to
// different warps) in a grid-strided order and runs two phases per batch.
//
//   Probe   one THREAD per (query, order): lane 4*ql + oi forms the key of the trailing
//           orders[oi]-gram of the batch's query ql, fetches both candidate buckets (64 bytes
//           each: two-choice cuckoo hashing, a key sits in one of the two) with four 32-byte
//           loads and scans them in registers.  A match of a hashed order is confirmed against
//           the stored tuple.
//           The four lanes of a query then agree on the retained phrase (LONGEST) or each keeps
//           its own (ALL); lane 4*ql records the result.
//   Gather  the whole warp per query: h streams to out in 16-byte vectors, GPU hits fetch their
//           row alongside and add g*m.
//
// Why a thread and not a group of lanes per probe: the probe is a few dozen instructions plus one
// dependent load.  A warp that spends its instruction slots on 4 probes at a time (8 lanes
// scanning one bucket, ballots and shuffles to combine) executed ~780 instructions per query and
// the call was issue-bound at 45 us; per-thread probing needs ~200.
// Why no block-wide phases: the longest probe chain among 256 threads (a run of full buckets) is
// several dependent DRAM round trips, and a barrier makes 8 warps wait for it (measured: 12.8 us
// of probing before any byte streamed).  Autonomous warps wait only for their own 32 lanes while
// the other warps of the SM keep the memory pipes busy.
#ifndef TFE_MIN_BLOCKS_GENERAL
#define TFE_MIN_BLOCKS_GENERAL 2     // blocks per SM the COSINE and the ALL variants are compiled for (the others: TFE_MIN_BLOCKS)
#endif
#ifndef TFE_MIN_BLOCKS
#define TFE_MIN_BLOCKS 3
#endif

template <int HT, bool ALL, bool COS, bool PACKED>
__global__ void __launch_bounds__(TFE_BLOCK_THREADS, (COS || ALL) ? TFE_MIN_BLOCKS_GENERAL : TFE_MIN_BLOCKS)
tfe_lookup_inject_kernel(const TfeLookupParams p)
{
    constexpr int VN = TfeVec<HT>::N;
    constexpr int UNROLL = 4;
    static_assert(!PACKED || (HT == 0 && !ALL && !COS), "packed bf16 path is LONGEST/CONST on bf16 only");

    const int lane = threadIdx.x & 31;
    const int cols = ALL ? p.n_orders : 1;
    const int steps = p.d / VN;                  // 16-byte steps of h per row
    const size_t hid_row_bytes = (size_t)p.d * (HT == 0 ? 2 : 4);
    const bool in_place = p.out == p.h;
    const int ql = lane >> 2, oi = lane & 3;
    const int my_order = oi < p.n_orders ? p.orders[oi] : 0;
    const bool my_hashed = my_order > 0 && !tfe_order_is_packed(my_order, p.tok_bits);
    const uint32_t qb = p.qb;
    const uint32_t n_batches = (p.Q + qb - 1) / qb;
    uint32_t my_miss = 0;                        // per thread here; summed per warp below

    __shared__ TfeProbeTick s_tick;
    if (threadIdx.x == 0) s_tick.warps_and_misses = 0ull;
    __syncthreads();
    tfe_grid_dependency_sync();
    const uint32_t tag = tfe_call_tag(p.counters);
    const uint32_t n_warps = gridDim.x * TFE_WARPS_PER_BLOCK;
    // ALL / CONST reports after its rows instead of after its last probe: with the report inside the
    // batch loop that instantiation measured 58.4 us on the 32,768-token prefill, 49.4 us this way
    // (the gated ones gained from the early report: LONGEST 35.4 -> 34.4 us, ALL decode 8.1 -> 6.5 us)
    constexpr bool LATE_TICK = ALL && !COS;
    if (!LATE_TICK && blockIdx.x * TFE_WARPS_PER_BLOCK + (threadIdx.x >> 5) >= n_batches) tfe_warp_probing_done(p, &s_tick, 0u);     // a warp without queries
    for (uint32_t batch = blockIdx.x * TFE_WARPS_PER_BLOCK + (threadIdx.x >> 5); batch < n_batches; batch += n_warps) {
        // query lq of batch b is b + lq * n_batches: the queries of a warp are spread over the call,
        // so a run of consecutive positions that all hit is shared out among many warps
        // ================================ probe phase ================================
        const uint32_t q = batch + (uint32_t)ql * n_batches;
        const bool mine = ql < (int)qb && q < p.Q;
        const unsigned long long found = tfe_probe_lane(p, q, mine, my_order, my_hashed);
        // ---- selection policy + tier walk; the 4 lanes of a query form one aligned quad
        __syncwarp();
        int32_t my_slot = -1;                    // GPU-tier slot this lane contributes, or -1
        float my_alpha = 0.f;
        if constexpr (!ALL) {
            my_slot = tfe_select_longest(p, found, q, mine, lane, my_miss, tag);
        } else {
            const uint32_t quad_found = (__ballot_sync(0xFFFFFFFFu, found != TFE_NONE64) >> (lane & ~3)) & 0xFu;
            int n_sum = 0;                       // sum of the matched orders of this query
#pragma unroll
            for (int g = 0; g < 4; ++g)
                if ((quad_found >> g) & 1u) n_sum += p.orders[g];
            if (oi < p.n_orders && mine) {
                uint32_t phrase = 0xFFFFFFFFu;
                int32_t st_ = -3;
                uint32_t flag = 0;
                if (found != TFE_NONE64) {
                    phrase = (uint32_t)(found >> 32);
                    st_ = (int32_t)(uint32_t)found;
                    flag = st_ >= 0 ? 1 : (st_ == -1 ? 2 : 3);
                }
                if (flag == 1) { my_slot = st_; my_alpha = (float)my_order / (float)n_sum; }
                const size_t k = (size_t)q * cols + oi;
                p.scr_rec[k] = tfe_make_record(tag, flag, phrase);
                if (flag >= 2) ++my_miss;
                if (p.flags) p.flags[k] = (uint8_t)flag;
                if (p.sel_phrase) p.sel_phrase[k] = phrase;
                if (p.sel_slot) p.sel_slot[k] = st_;
            }
        }

        if (p.slot_stats != nullptr && my_slot >= 0) tfe_touch_slot(p.slot_stats, my_slot, __ldcg(p.epoch));
        if (!LATE_TICK && batch + n_warps >= n_batches)        // this warp's last probe is on record: report (its rows are still to stream)
            tfe_warp_probing_done(p, &s_tick, __reduce_add_sync(0xFFFFFFFFu, my_miss));

        // ================================ gather phase ===============================
        for (uint32_t lq = 0; lq < qb; ++lq) {
            const uint32_t gq = batch + lq * n_batches;
            if (gq >= p.Q) break;
            const char *hrow = reinterpret_cast<const char *>(p.h) + (size_t)gq * hid_row_bytes;
            char *orow = reinterpret_cast<char *>(p.out) + (size_t)gq * hid_row_bytes;
            // rows to add: held by the lanes of quad lq
            const uint4 *rowp[ALL ? 4 : 1];
            float alpha[ALL ? 4 : 1];
            int n_rows = 0;
#pragma unroll
            for (int g = 0; g < (ALL ? 4 : 1); ++g) {
                const int32_t sl = __shfl_sync(0xFFFFFFFFu, my_slot, 4 * lq + g);
                alpha[g] = ALL ? __shfl_sync(0xFFFFFFFFu, my_alpha, 4 * lq + g) : 1.f;
                rowp[g] = sl >= 0 ? p.rows + (size_t)sl * (size_t)(p.d / 8) : nullptr;
                n_rows += sl >= 0;
            }
            if (n_rows == 0) {                   // nothing to add: out = h bit for bit
                if (!in_place) {
                    for (int s0 = 0; s0 < steps; s0 += 32 * UNROLL) {
                        uint4 v[UNROLL];
#pragma unroll
                        for (int u = 0; u < UNROLL; ++u) {
                            const int k = s0 + u * 32 + lane;
                            if (k < steps) v[u] = ld_stream(reinterpret_cast<const uint4 *>(hrow) + k);
                        }
#pragma unroll
                        for (int u = 0; u < UNROLL; ++u) {
                            const int k = s0 + u * 32 + lane;
                            if (k < steps) st_stream(reinterpret_cast<uint4 *>(orow) + k, v[u]);
                        }
                    }
                }
                continue;
            }
            float gate = p.lambda;
            if constexpr (COS && !ALL) {
                // a row of at most 32 * UNROLL steps stays in registers between the dot products
                // and the update: one trip to memory instead of two
                if (steps <= 32 * UNROLL) {
                    uint4 hv[UNROLL];
                    typename TfeVec<HT>::RowRaw rv[UNROLL];
#pragma unroll
                    for (int u = 0; u < UNROLL; ++u) {
                        const int k = u * 32 + lane;
                        if (k < steps) {
                            hv[u] = ld_stream(reinterpret_cast<const uint4 *>(hrow) + k);
                            rv[u] = ld_row_raw<HT>(rowp[0], k);
                        }
                    }
                    float sa = 0.f, sb = 0.f, sc = 0.f;      // <h,m>, <h,h>, <m,m>, same order of terms as below
#pragma unroll
                    for (int u = 0; u < UNROLL; ++u) {
                        if (u * 32 + lane >= steps) continue;
                        float x[VN], m[VN];
                        unpack_hidden<HT>(hv[u], x);
                        unpack_row<HT>(rv[u], m);
#pragma unroll
                        for (int e = 0; e < VN; ++e) {
                            sa = fmaf(x[e], m[e], sa); sb = fmaf(x[e], x[e], sb); sc = fmaf(m[e], m[e], sc);
                        }
                    }
                    sa = warp_sum(sa); sb = warp_sum(sb); sc = warp_sum(sc);
                    gate = p.lambda / (1.f + __expf(-sa * rsqrtf(fmaf(sb, sc, 1e-12f))));
#pragma unroll
                    for (int u = 0; u < UNROLL; ++u) {
                        const int k = u * 32 + lane;
                        if (k >= steps) continue;
                        float x[VN], m[VN], y[VN];
                        unpack_hidden<HT>(hv[u], x);
                        unpack_row<HT>(rv[u], m);
#pragma unroll
                        for (int e = 0; e < VN; ++e) y[e] = fmaf(gate, m[e], x[e]);
                        store_hidden<HT>(orow, k, y);
                    }
                    continue;
                }
            }
            if constexpr (ALL) {
                // every row of the query in flight together, the weighted sum m kept in registers: the rows are
                // read once (the gated form needs the whole of m before its update, so it takes this path only
                // when one trip covers the row)
                constexpr int UA = UNROLL;
                if (!COS || steps <= 32 * UA) {
                    for (int s0 = 0; s0 < steps; s0 += 32 * UA) {
                        uint4 hv[UA];
                        float m[UA][VN];
#pragma unroll
                        for (int u = 0; u < UA; ++u) {
                            const int k = s0 + u * 32 + lane;
                            if (k < steps) hv[u] = ld_stream(reinterpret_cast<const uint4 *>(hrow) + k);
#pragma unroll
                            for (int e = 0; e < VN; ++e) m[u][e] = 0.f;
                        }
#pragma unroll
                        for (int g = 0; g < 4; ++g) {
                            if (rowp[g] == nullptr) continue;
                            typename TfeVec<HT>::RowRaw rv[UA];
#pragma unroll
                            for (int u = 0; u < UA; ++u) {
                                const int k = s0 + u * 32 + lane;
                                if (k < steps) rv[u] = ld_row_raw<HT>(rowp[g], k);
                            }
#pragma unroll
                            for (int u = 0; u < UA; ++u) {
                                if (s0 + u * 32 + lane >= steps) continue;
                                float r[VN];
                                unpack_row<HT>(rv[u], r);
#pragma unroll
                                for (int e = 0; e < VN; ++e) m[u][e] = fmaf(alpha[g], r[e], m[u][e]);
                            }
                        }
                        if constexpr (COS) {
                            float sa = 0.f, sb = 0.f, sc = 0.f;      // <h,m>, <h,h>, <m,m>, same order of terms as below
#pragma unroll
                            for (int u = 0; u < UA; ++u) {
                                if (s0 + u * 32 + lane >= steps) continue;
                                float x[VN];
                                unpack_hidden<HT>(hv[u], x);
#pragma unroll
                                for (int e = 0; e < VN; ++e) {
                                    sa = fmaf(x[e], m[u][e], sa); sb = fmaf(x[e], x[e], sb); sc = fmaf(m[u][e], m[u][e], sc);
                                }
                            }
                            sa = warp_sum(sa); sb = warp_sum(sb); sc = warp_sum(sc);
                            gate = p.lambda / (1.f + __expf(-sa * rsqrtf(fmaf(sb, sc, 1e-12f))));
                        }
#pragma unroll
                        for (int u = 0; u < UA; ++u) {
                            const int k = s0 + u * 32 + lane;
                            if (k >= steps) continue;
                            float x[VN], y[VN];
                            unpack_hidden<HT>(hv[u], x);
#pragma unroll
                            for (int e = 0; e < VN; ++e) y[e] = fmaf(gate, m[u][e], x[e]);
                            store_hidden<HT>(orow, k, y);
                        }
                    }
                    continue;
                }
            }
            if constexpr (COS) {
                float sa = 0.f, sb = 0.f, sc = 0.f;      // <h,m>, <h,h>, <m,m>
#pragma unroll (COS ? 2 : 1)
                for (int k = lane; k < steps; k += 32) {
                    float x[VN], m[VN];
                    load_hidden<HT>(hrow, k, x);
                    load_memory<HT, ALL>(rowp, alpha, k, m);
#pragma unroll
                    for (int e = 0; e < VN; ++e) {
                        sa = fmaf(x[e], m[e], sa); sb = fmaf(x[e], x[e], sb); sc = fmaf(m[e], m[e], sc);
                    }
                }
                sa = warp_sum(sa); sb = warp_sum(sb); sc = warp_sum(sc);
                gate = p.lambda / (1.f + __expf(-sa * rsqrtf(fmaf(sb, sc, 1e-12f))));
            }
            if constexpr (!ALL) {
                // one row: keep the raw 16-byte vectors in flight, convert when they are consumed
                for (int s0 = 0; s0 < steps; s0 += 32 * UNROLL) {
                    uint4 hv[UNROLL];
                    typename TfeVec<HT>::RowRaw rv[UNROLL];
#pragma unroll
                    for (int u = 0; u < UNROLL; ++u) {
                        const int k = s0 + u * 32 + lane;
                        if (k < steps) {
                            hv[u] = ld_stream(reinterpret_cast<const uint4 *>(hrow) + k);
                            rv[u] = ld_row_raw<HT>(rowp[0], k);
                        }
                    }
#pragma unroll
                    for (int u = 0; u < UNROLL; ++u) {
                        const int k = s0 + u * 32 + lane;
                        if (k >= steps) continue;
                        if constexpr (PACKED) {
                            // lambda is a bf16 number: one fused multiply-add per bf16 pair, rounded
                            // once from the exact h + lambda*m
                            const uint32_t lam2 = p.lambda_bf16x2;
                            uint4 o;
                            o.x = fma_bf16x2(lam2, rv[u].x, hv[u].x); o.y = fma_bf16x2(lam2, rv[u].y, hv[u].y);
                            o.z = fma_bf16x2(lam2, rv[u].z, hv[u].z); o.w = fma_bf16x2(lam2, rv[u].w, hv[u].w);
                            st_stream(reinterpret_cast<uint4 *>(orow) + k, o);
                        } else {
                            float x[VN], m[VN], y[VN];
                            unpack_hidden<HT>(hv[u], x);
                            unpack_row<HT>(rv[u], m);
#pragma unroll
                            for (int e = 0; e < VN; ++e) y[e] = fmaf(gate, m[e], x[e]);
                            store_hidden<HT>(orow, k, y);
                        }
                    }
                }
            } else {
#pragma unroll (COS ? 2 : 1)
                for (int k = lane; k < steps; k += 32) {
                    float x[VN], m[VN], y[VN];
                    load_hidden<HT>(hrow, k, x);
                    load_memory<HT, ALL>(rowp, alpha, k, m);
#pragma unroll
                    for (int e = 0; e < VN; ++e) y[e] = fmaf(gate, m[e], x[e]);
                    store_hidden<HT>(orow, k, y);
                }
            }
        }
    }

    if (LATE_TICK) tfe_warp_probing_done(p, &s_tick, __reduce_add_sync(0xFFFFFFFFu, my_miss));
    tfe_closing_block_epilogue(p, cols, tag, true);
}

// ------------------------------------- the hot path, LONGEST / CONST version
//
// The same batches, the same two phases and bit-identical results as the general kernel above
// for the policy the benchmark grades.  A probe is shared by a PAIR of lanes: each loads one 32-byte half
// of both candidate buckets (two loads in flight per lane, 16 registers instead of 32 -- this is what
// keeps the kernel from spilling inside its 80 registers -- and the two halves of a bucket are one line,
// so the load unit handles half as many lines per probe), the pair then agrees by one exchange.  A query
// takes 2 * n_orders lanes (at least 4: the four ids an n-gram can need are fetched one per lane), so a
// batch holds up to 8 / 5 / 4 queries with <= 2 / 3 / 4 orders.  The probe's three dependent steps (token
// ids -> buckets -> stored tuple) are cut down to one exposed step per batch:
//   * the token ids of the NEXT batch are requested while the current batch streams (one id per
//     lane, shared inside the quad by shuffles), so a batch starts with its ids in registers;
//   * the stored tuple of a hashed-order match is requested but not waited for: selection runs on
//     the key matches, the loads of the batch's first row are issued, and only then is the tuple
//     compared and the selection made final and recorded.  A key match whose tuple differs (two
//     phrases with one 64-bit key cannot both be in the table, so this means the n-gram is not a
//     phrase) simply repeats the first row's loads with the corrected choice; nothing has been
//     stored before that point, in place or not.
// UNROLL: 16-byte vectors of h (and of the row) a lane holds at a time.  4: a 1,024-element row is in flight whole,
// 80 registers, three blocks per SM.  2: 64 registers, four blocks per SM -- for rows of several chunks, where
// a warp walks chunk after chunk and a third more warps pays (8 KB rows: 278 -> 254 us per 65,536-token call).
template <int HT, bool PACKED, bool RANGED, int UNROLL, bool COS = false>
__global__ void __launch_bounds__(TFE_BLOCK_THREADS, UNROLL == 4 ? TFE_MIN_BLOCKS : TFE_MIN_BLOCKS + 1)
tfe_lookup_inject_longest_kernel(const TfeLookupParams p)
{
    // COS: the gate lambda * sigmoid(cos(h, m)) instead of lambda.  The host uses it only for rows one trip covers
    // (at most 32 * UNROLL steps), so the row and the hidden state are in registers when the three dot products
    // are formed, and only without the packed arithmetic and without ranges.
    static_assert(!COS || (!PACKED && !RANGED && UNROLL == 4), "the gated form is one instantiation per hidden type");
    constexpr int VN = TfeVec<HT>::N;
    static_assert(!PACKED || HT == 0, "packed bf16 path needs bf16 hidden states");

    const int lane = threadIdx.x & 31;
    const int steps = p.d / VN;                  // 16-byte steps of h per row
    const size_t hid_row_bytes = (size_t)p.d * (HT == 0 ? 2 : 4);
    const bool in_place = p.out == p.h;
    const int lpq = max(4, 2 * p.n_orders);      // lanes per query
    const int ql = lane / lpq, role = lane - ql * lpq, base = ql * lpq;
    const int oi = role >> 1, half = role & 1;   // order column and bucket half of this lane's probe
    const int my_order = oi < p.n_orders ? p.orders[oi] : 0;
    const bool my_hashed = my_order > 0 && !tfe_order_is_packed(my_order, p.tok_bits);
    const uint32_t qb = p.qb;                    // <= 32 / lpq
    // RANGED: the call is issued in several launches, each over a query range [q_lo, q_hi)
    const uint32_t q_lo = RANGED ? p.q_lo : 0u, q_hi = RANGED ? p.q_hi : p.Q;
    // Work split: warp w of the launch owns the queries q_lo + w + k * n_warps, k = 0 .. cnt-1: every warp gets the
    // same number of queries to within one, neighbouring positions go to neighbouring warps (a run of consecutive
    // positions that all hit -- overlapping phrases -- is shared out among many warps, and the rows that are in
    // flight at one time lie close together).  A warp walks its queries in rounds of qb.
    const uint32_t n_warps = gridDim.x * TFE_WARPS_PER_BLOCK;
    const uint32_t q_first = q_lo + blockIdx.x * TFE_WARPS_PER_BLOCK + (threadIdx.x >> 5);
    const uint32_t cnt = q_first < q_hi ? (q_hi - q_first + n_warps - 1) / n_warps : 0u;
    __shared__ TfeProbeTick s_tick;
    if (threadIdx.x == 0) s_tick.warps_and_misses = 0ull;
    __syncthreads();
    tfe_grid_dependency_sync();
    const uint32_t tag = tfe_call_tag(p.counters);
    const uint32_t epoch = p.slot_stats != nullptr ? __ldcg(p.epoch) : 0u;
    uint32_t my_miss = 0;

    // the id `role` places before this lane's query of the round that starts at the warp's query k0 (roles 0..3),
    // or -1 (no such query / position / padding id)
    auto fetch_token = [&](uint32_t k0) -> int32_t {
        const uint32_t k = k0 + (uint32_t)ql;
        int32_t v = -1;
        if (ql < (int)qb && k < cnt && role < 4) {
            const uint32_t q = q_first + k * n_warps;
            const uint32_t b = tfe_div(q, p.div_tq);
            const int32_t t = p.q_start + (int32_t)(q - b * (uint32_t)p.Tq) - role;
            if (t >= 0) {
                v = __ldg(p.tokens + (size_t)b * p.T + t);
                if ((uint32_t)v >= (uint32_t)p.vocab) v = -1;
            }
        }
        return v;
    };
    // slot of the retained phrase if it is GPU-resident (valid on the query's first lane), else -1
    const uint32_t group_mask = (1u << lpq) - 1u;
    auto choose = [&](unsigned long long f) -> int32_t {
        const uint32_t group_found = (__ballot_sync(0xFFFFFFFFu, f != TFE_NONE64) >> base) & group_mask;
        const int top = group_found ? 31 - __clz(group_found) : 0;      // a lane of the greatest order that matched
        const unsigned long long sel = __shfl_sync(0xFFFFFFFFu, f, base + top);
        const int32_t st_ = (int32_t)(uint32_t)sel;
        return (role == 0 && group_found && st_ >= 0) ? st_ : -1;
    };

    if (cnt == 0) tfe_warp_probing_done(p, &s_tick, 0u);     // a warp without queries
    int32_t tok = fetch_token(0);
    for (uint32_t k0 = 0; k0 < cnt; k0 += qb) {
        const uint32_t q = q_first + (k0 + (uint32_t)ql) * n_warps;
        const bool mine = ql < (int)qb && k0 + (uint32_t)ql < cnt;

        // ================================ probe phase ================================
        int32_t tk[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) tk[j] = __shfl_sync(0xFFFFFFFFu, tok, base + j);
        tok = fetch_token(k0 + qb);              // lands while this round is processed
        bool ok = mine && my_order > 0;
#pragma unroll
        for (int j = 0; j < 4; ++j)
            if (j < my_order && tk[j] < 0) ok = false;
        unsigned long long found = TFE_NONE64;
        int4 tuple = make_int4(0, 0, 0, 0);
        if (ok) {
            const uint64_t key = tfe_make_key(my_order, tk, p.tok_bits);
            const uint64_t b1 = tfe_home_bucket_of(key, p.n_buckets);
            const uint64_t b2 = tfe_second_bucket_of(key, b1, p.n_buckets);
            const ulonglong4 *p1 = reinterpret_cast<const ulonglong4 *>(p.index + b1 * TFE_SLOTS_PER_BUCKET);
            const ulonglong4 *p2 = reinterpret_cast<const ulonglong4 *>(p.index + b2 * TFE_SLOTS_PER_BUCKET);
            ulonglong4 w[2];                     // this lane's half (2 slots of {key, value}) of both buckets, both loads in flight
            w[0] = ld_bucket32(p1 + half); w[1] = ld_bucket32(p2 + half);
#pragma unroll
            for (int k = 0; k < 2; ++k) {
                if (w[k].x == key) found = w[k].y;
                if (w[k].z == key) found = w[k].w;
            }
        }
        __syncwarp();
        {   // the pair agrees: the key sits in at most one slot, "none" is the largest value
            const unsigned long long other = __shfl_xor_sync(0xFFFFFFFFu, found, 1);
            found = other < found ? other : found;
        }
        if (my_hashed && found != TFE_NONE64) tuple = __ldg(p.phrase_tokens + (uint32_t)(found >> 32));
        const int32_t guess = choose(found);     // selection on key matches, tuples not yet compared

        // ---- loads of the batch's first row, issued on the guess
        uint4 hv[UNROLL];
        typename TfeVec<HT>::RowRaw rv[UNROLL];
        auto issue_first = [&](uint32_t lq, int32_t sl) {
            const char *hrow = reinterpret_cast<const char *>(p.h) + (size_t)(q_first + (k0 + lq) * n_warps) * hid_row_bytes;
            const uint4 *rowp = p.rows + (size_t)(sl >= 0 ? sl : 0) * (size_t)(p.d / 8);
            if (sl >= 0 || !in_place) {
#pragma unroll
                for (int u = 0; u < UNROLL; ++u) {
                    const int k = u * 32 + lane;
                    if (k < steps) {
                        hv[u] = ld_stream(reinterpret_cast<const uint4 *>(hrow) + k);
                        if (sl >= 0) rv[u] = ld_row_raw<HT>(rowp, k);
                    }
                }
            }
        };
        const int32_t guess0 = __shfl_sync(0xFFFFFFFFu, guess, 0);
        issue_first(0, guess0);

        // ---- the tuples have arrived by now: final selection, tier walk, record
        if (my_hashed && found != TFE_NONE64 && !tuple_matches(tuple, tk, my_order)) found = TFE_NONE64;
        const int32_t my_slot = tfe_select_longest_group(p, found, q, mine, base, group_mask, role == 0, my_miss, tag);
        const bool redo_first = __shfl_sync(0xFFFFFFFFu, my_slot, 0) != guess0;
        if (k0 + qb >= cnt)                      // this warp's last probe is on record: report (its rows are still to stream)
            tfe_warp_probing_done(p, &s_tick, __reduce_add_sync(0xFFFFFFFFu, my_miss));

        // ================================ gather phase ===============================
        const uint32_t n_round = min(qb, cnt - k0);
        for (uint32_t lq = 0; lq < n_round; ++lq) {
            const uint32_t gq = q_first + (k0 + lq) * n_warps;
            const int32_t sl = __shfl_sync(0xFFFFFFFFu, my_slot, lpq * (int)lq);
            if (lq > 0 || redo_first) issue_first(lq, sl);
            if (sl < 0 && in_place) continue;    // nothing to add and nothing to copy
            const char *hrow = reinterpret_cast<const char *>(p.h) + (size_t)gq * hid_row_bytes;
            char *orow = reinterpret_cast<char *>(p.out) + (size_t)gq * hid_row_bytes;
            const uint4 *rowp = p.rows + (size_t)(sl >= 0 ? sl : 0) * (size_t)(p.d / 8);
            for (int s0 = 0; s0 < steps; s0 += 32 * UNROLL) {
                if (s0 > 0) {
#pragma unroll
                    for (int u = 0; u < UNROLL; ++u) {
                        const int k = s0 + u * 32 + lane;
                        if (k < steps) {
                            hv[u] = ld_stream(reinterpret_cast<const uint4 *>(hrow) + k);
                            if (sl >= 0) rv[u] = ld_row_raw<HT>(rowp, k);
                        }
                    }
                }
                float gate = p.lambda;
                if constexpr (COS) {
                    if (sl >= 0) {
                        float sa = 0.f, sb = 0.f, sc = 0.f;      // <h,m>, <h,h>, <m,m>: the general kernel's order of terms
#pragma unroll
                        for (int u = 0; u < UNROLL; ++u) {
                            if (u * 32 + lane >= steps) continue;
                            float x[VN], m[VN];
                            unpack_hidden<HT>(hv[u], x);
                            unpack_row<HT>(rv[u], m);
#pragma unroll
                            for (int e = 0; e < VN; ++e) {
                                sa = fmaf(x[e], m[e], sa); sb = fmaf(x[e], x[e], sb); sc = fmaf(m[e], m[e], sc);
                            }
                        }
                        sa = warp_sum(sa); sb = warp_sum(sb); sc = warp_sum(sc);
                        gate = p.lambda / (1.f + __expf(-sa * rsqrtf(fmaf(sb, sc, 1e-12f))));
                    }
                }
#pragma unroll
                for (int u = 0; u < UNROLL; ++u) {
                    const int k = s0 + u * 32 + lane;
                    if (k >= steps) continue;
                    if (sl < 0) {                // out = h bit for bit
                        st_stream(reinterpret_cast<uint4 *>(orow) + k, hv[u]);
                    } else if constexpr (PACKED) {
                        // lambda is a bf16 number: one fused multiply-add per bf16 pair, rounded once
                        // from the exact h + lambda*m
                        const uint32_t lam2 = p.lambda_bf16x2;
                        uint4 o;
                        o.x = fma_bf16x2(lam2, rv[u].x, hv[u].x); o.y = fma_bf16x2(lam2, rv[u].y, hv[u].y);
                        o.z = fma_bf16x2(lam2, rv[u].z, hv[u].z); o.w = fma_bf16x2(lam2, rv[u].w, hv[u].w);
                        st_stream(reinterpret_cast<uint4 *>(orow) + k, o);
                    } else {
                        float x[VN], m[VN], y[VN];
                        unpack_hidden<HT>(hv[u], x);
                        unpack_row<HT>(rv[u], m);
#pragma unroll
                        for (int e = 0; e < VN; ++e) y[e] = fmaf(gate, m[e], x[e]);
                        store_hidden<HT>(orow, k, y);
                    }
                }
            }
        }
        // bookkeeping for the retention ranking, off the path between probe and gather
        if (p.slot_stats != nullptr && my_slot >= 0) tfe_touch_slot(p.slot_stats, my_slot, epoch);
    }

    tfe_closing_block_epilogue(p, 1, tag, !RANGED || p.finalize != 0);
}

// ------------------------------------------------------------ streaming copy
//
// A plain grid-stride copy with the instructions the lookup kernels stream hidden states with; the benchmark's
// yardstick for "what a copy of this many bytes reaches".
__global__ void __launch_bounds__(256) tfe_stream_copy_kernel(const uint4 *__restrict__ src, uint4 *__restrict__ dst, size_t n)
{
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    for (; i + 3 * stride < n; i += 4 * stride) {
        const uint4 v0 = ld_stream(src + i), v1 = ld_stream(src + i + stride), v2 = ld_stream(src + i + 2 * stride),
                    v3 = ld_stream(src + i + 3 * stride);
        st_stream(dst + i, v0); st_stream(dst + i + stride, v1); st_stream(dst + i + 2 * stride, v2);
        st_stream(dst + i + 3 * stride, v3);
    }
    for (; i < n; i += stride) st_stream(dst + i, ld_stream(src + i));
}

// ------------------------------------------------------------- cache install

// One warp per installed row: the previous owner of the slot falls back to the
// host tier, the row is copied in, the phrase's index value becomes {id, slot}.
__global__ void __launch_bounds__(TFE_BLOCK_THREADS)
tfe_install_kernel(ulonglong2 *index, const uint32_t *phrase_pos, uint32_t *slot_owner, uint4 *rows,
                   int32_t row_vecs, int32_t n, const uint32_t *ids, const uint4 *src,
                   const int32_t *dst_slots, uint2 *slot_stats, const uint32_t *epoch)
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
        if (slot_stats != nullptr) slot_stats[dst] = make_uint2(1u, *epoch);     // used once, now
    }
    const uint4 *s = src + (size_t)k * row_vecs;
    uint4 *o = rows + (size_t)dst * row_vecs;
    for (int i = lane; i < row_vecs; i += 32) o[i] = ld_stream(s + i);
}

// ---------------------------------------------- cache install from the device
//
// The same insertion for a batch that lives on the device and was never checked by the host (the
// output of the candidate step and of the victim selection): entries that cannot be applied are
// skipped.  Judged against the state before the call, entry k is a candidate if its id is a
// phrase, the phrase is not GPU-resident, its slot exists and no earlier entry names the same
// phrase; it is applied if, in addition, no earlier candidate names the same slot.  "Earlier" is
// settled with one atomicMax per entry on a stamp per phrase and per slot: the stamp of entry k is
// 4096 - k, so the smallest k wins; the stamps are zero between calls (the last kernel puts back the
// ones this call touched), so the call keeps no state on the host and can be replayed from a graph.
//
//   tfe_install_claim_kernel     ONE block (a batch is at most 4,096 entries, four per thread), four steps with a
//                                block barrier between them: every entry stamps its phrase; every candidate stamps
//                                its slot; every entry learns whether it won both (flag, count); the stamps this
//                                call wrote go back to zero
//   tfe_install_device_kernel    one warp per entry: the winners install (as tfe_install_kernel)
#define TFE_INSTALL_DEVICE_MAX 4096

struct TfeInstallDeviceParams {
    ulonglong2 *index;
    const uint32_t *phrase_pos;
    uint32_t *slot_owner;
    uint4 *rows;
    int32_t row_vecs;
    int32_t n;
    uint32_t n_phrases;
    int64_t gpu_slots;
    const uint32_t *ids;            // [n]
    const uint4 *src;               // [n][row_vecs]
    const int32_t *dst_slots;       // [n]
    uint32_t *phrase_stamp;         // [n_phrases]
    uint32_t *slot_stamp;           // [gpu_slots]
    uint8_t *applied;               // [n] or nullptr
    uint8_t *flags;                 // [TFE_INSTALL_DEVICE_MAX] the same, owned by the context: claim kernel -> install kernel
    uint32_t *count;                // entries applied (written by the claim kernel)
    uint2 *slot_stats;
    const uint32_t *epoch;
};

#define TFE_INSTALL_CLAIM_THREADS 1024

__global__ void __launch_bounds__(TFE_INSTALL_CLAIM_THREADS)
tfe_install_claim_kernel(const TfeInstallDeviceParams p)
{
    constexpr int PER = TFE_INSTALL_DEVICE_MAX / TFE_INSTALL_CLAIM_THREADS;
    __shared__ uint32_t s_warp[TFE_INSTALL_CLAIM_THREADS / 32];
    tfe_grid_dependency_sync();
    uint32_t id[PER];
    int32_t dst[PER];
    bool valid[PER], cand[PER];
    // ---- every entry stamps its phrase: 4096 - k, so the smallest k wins (never the cleared value 0)
#pragma unroll
    for (int j = 0; j < PER; ++j) {
        const int k = j * TFE_INSTALL_CLAIM_THREADS + threadIdx.x;
        valid[j] = false; id[j] = 0; dst[j] = -1;
        if (k < p.n) {
            id[j] = p.ids[k];
            dst[j] = p.dst_slots[k];
            valid[j] = id[j] < p.n_phrases;
            if (valid[j]) atomicMax(p.phrase_stamp + id[j], (uint32_t)(TFE_INSTALL_DEVICE_MAX - k));
        }
    }
    __syncthreads();
    // ---- every candidate stamps its slot
#pragma unroll
    for (int j = 0; j < PER; ++j) {
        const int k = j * TFE_INSTALL_CLAIM_THREADS + threadIdx.x;
        cand[j] = valid[j] && dst[j] >= 0 && (int64_t)dst[j] < p.gpu_slots &&
                  (int32_t)(uint32_t)p.index[p.phrase_pos[id[j]]].y < 0 &&                  // not resident before the call
                  __ldcg(p.phrase_stamp + id[j]) == (uint32_t)(TFE_INSTALL_DEVICE_MAX - k);
        if (cand[j]) atomicMax(p.slot_stamp + dst[j], (uint32_t)(TFE_INSTALL_DEVICE_MAX - k));
    }
    __syncthreads();
    // ---- who won both
    uint32_t mine = 0;
#pragma unroll
    for (int j = 0; j < PER; ++j) {
        const int k = j * TFE_INSTALL_CLAIM_THREADS + threadIdx.x;
        if (k >= p.n) continue;
        const bool apply = cand[j] && __ldcg(p.slot_stamp + dst[j]) == (uint32_t)(TFE_INSTALL_DEVICE_MAX - k);
        p.flags[k] = apply ? 1 : 0;
        if (p.applied) p.applied[k] = apply ? 1 : 0;
        mine += apply;
    }
    mine = __reduce_add_sync(0xFFFFFFFFu, mine);
    if ((threadIdx.x & 31) == 0) s_warp[threadIdx.x >> 5] = mine;
    __syncthreads();
    if (threadIdx.x == 0) {
        uint32_t total = 0;
        for (int w = 0; w < TFE_INSTALL_CLAIM_THREADS / 32; ++w) total += s_warp[w];
        *p.count = total;
    }
    // ---- the stamps go back to zero (every thread is past its last look at them)
#pragma unroll
    for (int j = 0; j < PER; ++j) {
        if (valid[j]) p.phrase_stamp[id[j]] = 0;
        if (dst[j] >= 0 && (int64_t)dst[j] < p.gpu_slots) p.slot_stamp[dst[j]] = 0;
    }
}

__global__ void __launch_bounds__(TFE_BLOCK_THREADS)
tfe_install_device_kernel(const TfeInstallDeviceParams p)
{
    tfe_grid_dependency_sync();
    const int lane = threadIdx.x & 31;
    const int k = blockIdx.x * TFE_WARPS_PER_BLOCK + (threadIdx.x >> 5);
    if (k >= p.n) return;
    if (__ldcg(p.flags + k) == 0) return;
    const uint32_t id = p.ids[k];
    const int32_t dst = p.dst_slots[k];
    if (lane == 0) {
        const uint32_t prev = p.slot_owner[dst];
        if (prev != 0xFFFFFFFFu)
            p.index[p.phrase_pos[prev]].y = ((unsigned long long)prev << 32) | 0xFFFFFFFFull;   // -1: host tier
        p.index[p.phrase_pos[id]].y = ((unsigned long long)id << 32) | (uint32_t)dst;
        p.slot_owner[dst] = id;
        if (p.slot_stats != nullptr) p.slot_stats[dst] = make_uint2(1u, *p.epoch);
    }
    const uint4 *s = p.src + (size_t)k * p.row_vecs;
    uint4 *o = p.rows + (size_t)dst * p.row_vecs;
    for (int i = lane; i < p.row_vecs; i += 32) o[i] = ld_stream(s + i);
}

// ------------------------------------------- prefetch candidates + priority
//
// Early-exit guided prefetching after the top-K tokens are known: every predicted next token is
// combined with the recent history of its sequence into the n-grams it would complete, those are
// looked up with the same probe as above, and every phrase found outside the GPU tier becomes a
// candidate with priority s = p * r * c (token probability, usefulness of the entry, benefit of
// fetching it from its tier).  The `budget` best are returned in descending priority.
//
//   tfe_prefetch_probe_kernel   one thread per (sequence, token, order): probe, score, append
//                               {priority, entry index} as one 64-bit key to a compact list
//   tfe_prefetch_select_kernel  one block: radix-select the budget-th largest key, gather the keys at
//                               or above it in shared memory, bitonic sort, write the result
// The priority is a non-negative fp32 number, so its bit pattern orders like its value; the low
// word of a key is ~index, so a descending key sort is descending priority with ascending
// (sequence, token, order) among equals, and keys are unique.
#define TFE_PREFETCH_MAX_BUDGET 4096

struct TfePrefetchParams {
    const int32_t *history;         // [B][H]
    const int32_t *cand;            // [B][K]
    const float *prob;              // [B][K]
    const float *usefulness;        // [N] or nullptr (= 1)
    int32_t B, H, K;
    uint32_t n_entries;             // B * K * n_orders
    TfeFastDiv div_orders, div_k;
    const ulonglong2 *index;
    uint64_t n_buckets;
    const int4 *phrase_tokens;
    int32_t n_orders, orders[4], tok_bits, vocab;
    float benefit_host, benefit_ssd;
    unsigned long long *keys;       // [n_entries] compact candidate list
    uint32_t *entry_phrase;         // [n_entries] by entry index
    uint8_t *entry_tier;
    uint32_t *counter;              // number of candidates (reset by the select kernel)
};

__global__ void __launch_bounds__(256) tfe_prefetch_probe_kernel(const TfePrefetchParams p)
{
    tfe_grid_dependency_sync();
    const uint32_t idx = blockIdx.x * blockDim.x + threadIdx.x;
    const int lane = threadIdx.x & 31;
    unsigned long long key64 = 0;
    if (idx < p.n_entries) {
        const uint32_t bk = tfe_div(idx, p.div_orders);
        const int oi = (int)(idx - bk * (uint32_t)p.n_orders);
        const uint32_t b = tfe_div(bk, p.div_k);
        const int n = p.orders[oi];
        int32_t tk[4] = {-1, -1, -1, -1};
        bool ok = n - 1 <= p.H;
        if (ok) {
            tk[0] = __ldg(p.cand + bk);
#pragma unroll
            for (int j = 1; j < 4; ++j)
                if (j < n) tk[j] = __ldg(p.history + (size_t)b * p.H + (p.H - j));
#pragma unroll
            for (int j = 0; j < 4; ++j)
                if (j < n && (uint32_t)tk[j] >= (uint32_t)p.vocab) ok = false;
        }
        if (ok) {
            const uint64_t key = tfe_make_key(n, tk, p.tok_bits);
            const uint64_t b1 = tfe_home_bucket_of(key, p.n_buckets);
            const uint64_t b2 = tfe_second_bucket_of(key, b1, p.n_buckets);
            const ulonglong4 *p1 = reinterpret_cast<const ulonglong4 *>(p.index + b1 * TFE_SLOTS_PER_BUCKET);
            const ulonglong4 *p2 = reinterpret_cast<const ulonglong4 *>(p.index + b2 * TFE_SLOTS_PER_BUCKET);
            ulonglong4 w[4];
            w[0] = ld_bucket32(p1); w[1] = ld_bucket32(p1 + 1);
            w[2] = ld_bucket32(p2); w[3] = ld_bucket32(p2 + 1);
            unsigned long long found = TFE_NONE64;
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                if (w[k].x == key) found = w[k].y;
                if (w[k].z == key) found = w[k].w;
            }
            if (found != TFE_NONE64 && !tfe_order_is_packed(n, p.tok_bits)) {
                const int4 st = __ldg(p.phrase_tokens + (uint32_t)(found >> 32));
                if (!tuple_matches(st, tk, n)) found = TFE_NONE64;
            }
            const int32_t state = (int32_t)(uint32_t)found;
            if (found != TFE_NONE64 && state < 0) {          // a phrase, and not in the GPU tier
                const uint32_t phrase = (uint32_t)(found >> 32);
                const float c = state == -1 ? p.benefit_host : p.benefit_ssd;
                const float r = p.usefulness ? __ldg(p.usefulness + phrase) : 1.f;
                const float s = __fmul_rn(__fmul_rn(__ldg(p.prob + bk), r), c);
                if (s > 0.f) {
                    key64 = ((unsigned long long)__float_as_uint(s) << 32) | (0xFFFFFFFFu - idx);
                    p.entry_phrase[idx] = phrase;
                    p.entry_tier[idx] = state == -1 ? 2 : 3;
                }
            }
        }
    }
    // append: one atomic per warp
    const uint32_t has = __ballot_sync(0xFFFFFFFFu, key64 != 0);
    if (has) {
        uint32_t base = 0;
        if (lane == __ffs(has) - 1) base = atomicAdd(p.counter, __popc(has));
        base = __shfl_sync(0xFFFFFFFFu, base, __ffs(has) - 1);
        if (key64 != 0) p.keys[base + __popc(has & ((1u << lane) - 1u))] = key64;
    }
}

__global__ void __launch_bounds__(1024)
tfe_prefetch_select_kernel(const unsigned long long *keys, const uint32_t *entry_phrase, const uint8_t *entry_tier,
                           uint32_t *counter, uint32_t budget, TfeFastDiv div_orders, uint32_t n_orders,
                           uint32_t *out_phrase, uint8_t *out_tier, float *out_score, uint32_t *out_src,
                           uint32_t *out_count)
{
    __shared__ unsigned long long s_keys[TFE_PREFETCH_MAX_BUDGET];
    __shared__ uint32_t s_hist[256];
    __shared__ uint32_t s_fill;
    __shared__ unsigned long long s_prefix;
    __shared__ uint32_t s_want;
    tfe_grid_dependency_sync();
    const uint32_t n = *(volatile uint32_t *)counter;
    const uint32_t take = min(n, budget);
    // ---- threshold: the take-th largest key, by most-significant-digit-first radix selection
    unsigned long long thresh = 0;
    if (n > take) {
        if (threadIdx.x == 0) { s_prefix = 0; s_want = take; }
        __syncthreads();
        for (int shift = 56; shift >= 0; shift -= 8) {
            if (threadIdx.x < 256) s_hist[threadIdx.x] = 0;
            __syncthreads();
            const unsigned long long prefix = s_prefix;
            const unsigned long long mask = shift == 56 ? 0ull : ~0ull << (shift + 8);
            for (uint32_t i = threadIdx.x; i < n; i += blockDim.x) {
                const unsigned long long k = keys[i];
                if ((k & mask) == prefix) atomicAdd(&s_hist[(k >> shift) & 0xFFu], 1u);
            }
            __syncthreads();
            if (threadIdx.x == 0) {
                uint32_t want = s_want, d = 255;
                for (;; --d) {               // digits from the top until `want` keys are covered
                    if (s_hist[d] >= want) break;
                    want -= s_hist[d];
                    if (d == 0) break;
                }
                s_want = want;
                s_prefix = prefix | ((unsigned long long)d << shift);
            }
            __syncthreads();
        }
        thresh = s_prefix;
    }
    // ---- gather the keys at or above the threshold (exactly `take`: keys are unique), pad, sort
    uint32_t pow2 = 1;
    while (pow2 < take) pow2 <<= 1;
    if (threadIdx.x == 0) s_fill = 0;
    for (uint32_t i = threadIdx.x; i < pow2; i += blockDim.x) s_keys[i] = 0;
    __syncthreads();
    for (uint32_t i = threadIdx.x; i < n; i += blockDim.x) {
        const unsigned long long k = keys[i];
        if (k >= thresh) s_keys[atomicAdd(&s_fill, 1u)] = k;
    }
    __syncthreads();
    for (uint32_t size = 2; size <= pow2; size <<= 1)
        for (uint32_t stride = size >> 1; stride > 0; stride >>= 1) {
            for (uint32_t i = threadIdx.x; i < pow2 / 2; i += blockDim.x) {
                const uint32_t lo = 2 * i - (i & (stride - 1));       // pairs (lo, lo + stride)
                const uint32_t hi = lo + stride;
                const bool descending = (lo & size) == 0;
                const unsigned long long a = s_keys[lo], b = s_keys[hi];
                if ((a < b) == descending) { s_keys[lo] = b; s_keys[hi] = a; }
            }
            __syncthreads();
        }
    for (uint32_t i = threadIdx.x; i < take; i += blockDim.x) {
        const unsigned long long k = s_keys[i];
        const uint32_t idx = 0xFFFFFFFFu - (uint32_t)k;
        out_phrase[i] = entry_phrase[idx];
        out_tier[i] = entry_tier[idx];
        out_score[i] = __uint_as_float((uint32_t)(k >> 32));
        out_src[i] = tfe_div(idx, div_orders);
    }
    // the rest of the budget names no phrase, so that the arrays can go to tfe_cache_install_device whole
    for (uint32_t i = take + threadIdx.x; i < budget; i += blockDim.x) out_phrase[i] = 0xFFFFFFFFu;
    __syncthreads();
    if (threadIdx.x == 0) {
        out_count[0] = take;
        out_count[1] = n;
        *counter = 0;                        // ready for the next call
    }
    (void)n_orders;
}



// ------------------------------------------------ GPU-tier retention ranking
//
// Which slots to overwrite next (Sec. 4.3: cached entries are ranked by access frequency and
// recency, among other signals; the formula is this library's).  Per slot the lookup kernels keep
// {freq, last}: injections served since the row was installed and the epoch (lookup count) of the
// most recent one.  At epoch `now`
//     age = now - last,  decayed = freq >> min(31, age / half_life)   (half_life <= 0: no decay)
//     key = min(decayed, 65535) << 16 | (65535 - min(age, 65535)),    0 for a slot without owner
// and the victims are the n slots of smallest (key, slot).  (key << 32 | slot) is a distinct
// 64-bit number per slot, so this is a selection of the n smallest of C distinct numbers, and it is
// ONE cooperative launch (tfe_victim_select_kernel, one block per SM) that reads the 8 bytes of
// bookkeeping per slot once (a slot without owner is marked in its freq word):
//
//   threshold   block 0 draws up to 2,048 slots, one from each of as many equal stretches of the table, and
//               publishes a threshold T that r or more of their numbers do not exceed; r sits six standard
//               deviations above the expected rank of the n-th smallest in the sample, so that n or more of
//               all numbers are <= T, but not many more (c4: ~90,000 of 16.8 M).  A table that fits the final
//               step whole skips this (T = max).
//   scan        the one pass over {freq, last}: every number <= T goes to a candidate list (collected per
//               block in shared memory, handed over with one atomic per 1,024) and is counted by its distance
//               below T on a logarithmic scale, 128 steps per octave.
//   narrow      from those counts: the piece of the scale that holds the n-th smallest, and how many numbers
//               lie beyond it.  Mostly the piece holds few enough to go on; else
//   refine      a histogram of the candidates over 2,048 equal parts of the piece, the part that holds the
//               n-th smallest becomes the new piece; repeated while it is too full.
//   final       everything up to the piece's upper end is gathered (n plus at most a few thousand numbers),
//               every block copies the set to shared memory and its warps place one number each by counting
//               the smaller ones; ranks below n are the result, already sorted.
//
// The result never depends on the sample: if fewer than n numbers turn out to be <= T, or more than the
// list holds, the later steps walk the table itself instead of the list (slower, same answer).
// Blocks wait for one another at the step boundaries (a counter in global memory, release / acquire); the
// launch is cooperative, so they are resident together, and every wait is bounded.
#define TFE_VICTIMS_MAX 4096
#define TFE_VS_THREADS 1024
#define TFE_VS_BINS 2048
#define TFE_VS_LIST_CAP (1024 * 1024)    // candidate list entries (8 MiB): the sampled threshold admits ~7 * C / 2,048 or more
#define TFE_VS_FINAL_CAP 8192            // most numbers the final step ranks; also the shared-memory buffer's entries
#define TFE_VS_FINAL_DEFAULT 5120        // refine until this many are left to rank ...
#define TFE_VS_RANGE_DEFAULT 2048        // ... or this many above the ones that are certain
#define TFE_VS_SAMPLES 2048
#define TFE_VS_MAX_REFINE 8              // a refine step shrinks hi - lo at least 1,024-fold: 7 cover 64 bits
#define TFE_VS_DYN_SMEM (TFE_VS_FINAL_CAP * 8)
#define TFE_VS_NEAR_MANT 7                                   // bits of T - number kept below its leading one
#define TFE_VS_NEAR_BINS ((64 - TFE_VS_NEAR_MANT + 1) << TFE_VS_NEAR_MANT)      // 7,424

#define TFE_VS_ERR_BARRIER 1u            // a wait at a step boundary ran out
#define TFE_VS_ERR_INTERNAL 2u           // counts that contradict one another

// All zero before a launch.  A launch that completes leaves it so (its blocks clear what they used once nobody
// reads it any more); one that gave up leaves `status` set and the rest as it was: the host clears it.
struct TfeVictimState {
    uint32_t arrived;               // blocks through the step boundaries so far
    uint32_t n_cand;                // numbers <= T seen by the scan (entries beyond the list's capacity are dropped)
    uint32_t n_final;               // numbers gathered for the final step
    uint32_t status;                // TFE_VS_ERR_*
    uint32_t threshold_ready;       // block 0 has published `threshold`
    uint32_t left;                  // blocks that have finished; the last one clears the counters for the next launch
    unsigned long long threshold;
    uint32_t near[TFE_VS_NEAR_BINS];   // candidates by tfe_vs_near_bin(T - number)
    uint32_t hist[TFE_VS_MAX_REFINE][TFE_VS_BINS];
};

struct TfeVictimParams {
    const uint2 *slot_stats;        // [C4] {freq, last}; freq = TFE_FREE_SLOT_FREQ marks a slot without owner
    const uint32_t *epoch;
    TfeFastDiv div_half_life;       // for half_life > 0 ...
    uint32_t age_cap;               // ... with 32 * half_life
    uint32_t C, take;
    uint32_t n_samples, sample_rank;    // 0 samples: no threshold
    uint32_t sample_stretch, sample_longer;     // C / n_samples, C % n_samples
    uint32_t list_cap, final_cap, range_cap;    // refine until <= final_cap numbers are left to rank, or <= range_cap above the certain ones
    unsigned long long *list;       // [list_cap]
    unsigned long long *fin;        // [TFE_VS_FINAL_CAP]
    TfeVictimState *st;
    int32_t *out_slots;             // [take]
    uint32_t *out_keys;             // [take]
};

// A slot without owner carries freq = TFE_FREE_SLOT_FREQ in its bookkeeping (written when the policy is enabled;
// a slot only ever goes from free to owned, and the installation overwrites the mark), so the ranking reads the
// 8 bytes of {freq, last} per slot and nothing else.
#define TFE_FREE_SLOT_FREQ 0xFFFFFFFFu
#define TFE_HALF_LIFE_MAX ((1 << 26) - 1)       // 32 * half_life stays below 2^31

__global__ void __launch_bounds__(256) tfe_policy_reset_kernel(uint2 *slot_stats, const uint32_t *slot_owner, uint32_t C)
{
    for (uint32_t i = blockIdx.x * blockDim.x + threadIdx.x; i < C; i += gridDim.x * blockDim.x)
        slot_stats[i] = make_uint2(slot_owner[i] == 0xFFFFFFFFu ? TFE_FREE_SLOT_FREQ : 0u, 0u);
}

// DECAY: half_life > 0.  age_cap = 32 * half_life (below 2^31, which the fast division needs): the quotient
// saturates at 31 from there on.
template <bool DECAY>
__device__ __forceinline__ uint32_t tfe_retention_key(uint2 st, uint32_t now, TfeFastDiv div, uint32_t age_cap)
{
    const uint32_t age = now - st.y;
    uint32_t decayed = st.x;
    if (DECAY) decayed >>= min(31u, tfe_div(min(age, age_cap), div));
    const uint32_t key = (min(decayed, 65535u) << 16) | (65535u - min(age, 65535u));
    return st.x == TFE_FREE_SLOT_FREQ ? 0u : key;
}

#define TFE_VS_NONE 0xFFFFFFFFFFFFFFFFull       // never a slot's number: slots are below 2^31

// Distance d = T - number of a candidate on a logarithmic scale with 128 steps per octave: d itself below 128,
// else the position of its leading one and the seven bits after it.  Grows with d; bin b >= 128 covers
// [m << s, ((m + 1) << s) - 1] with m = 128 + (b & 127), s = (b >> 7) - 1.
__device__ __forceinline__ uint32_t tfe_vs_near_bin(unsigned long long d)
{
    if (d < (1ull << TFE_VS_NEAR_MANT)) return (uint32_t)d;
    const int s = (63 - __clzll((long long)d)) - TFE_VS_NEAR_MANT;
    return ((uint32_t)(s + 1) << TFE_VS_NEAR_MANT) | ((uint32_t)(d >> s) & ((1u << TFE_VS_NEAR_MANT) - 1u));
}
__device__ __forceinline__ void tfe_vs_near_range(uint32_t b, unsigned long long &d_min, unsigned long long &d_max)
{
    if (b < (1u << TFE_VS_NEAR_MANT)) { d_min = d_max = b; return; }
    const int s = (int)(b >> TFE_VS_NEAR_MANT) - 1;
    const unsigned long long m = (1ull << TFE_VS_NEAR_MANT) | (b & ((1u << TFE_VS_NEAR_MANT) - 1u));
    d_min = m << s;
    d_max = d_min + ((1ull << s) - 1ull);
}

// Blocks of the launch meet: the b-th boundary is passed when b * gridDim.x arrivals are on record.
// False when the wait ran out or another block has reported an error (the caller returns at once).
__device__ __forceinline__ bool tfe_vs_boundary(TfeVictimState *st, uint32_t &boundary)
{
    __shared__ uint32_t s_ok;
    ++boundary;
    __syncthreads();
    if (threadIdx.x == 0) {
        // release: the block's writes (ordered before this thread by the barrier above) are visible to whoever
        // acquires the count
        asm volatile("red.release.gpu.global.add.u32 [%0], 1;" :: "l"(&st->arrived) : "memory");
        const uint32_t want = boundary * gridDim.x;
        const volatile uint32_t *status = &st->status;
        uint32_t spin = 0, seen = 0;
        bool ok = true;
        for (;;) {
            asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(seen) : "l"(&st->arrived) : "memory");
            if (seen >= want) break;
            if (*status != 0u || ++spin > TFE_SPIN_LIMIT) { ok = false; break; }
        }
        if (!ok) atomicOr(&st->status, TFE_VS_ERR_BARRIER);
        s_ok = ok;
    }
    __syncthreads();
    return s_ok != 0u;
}

// Numbers found by the threads of a block, collected in shared memory and handed to a global list with one
// atomic per 1,024 of them; a warp that finds many at once (a dense stretch) reserves in the global list directly.
struct TfeVsAppender {
    unsigned long long *buf;        // shared memory, `cap` entries, all TFE_VS_NONE before the first append
    uint32_t *s_count;              // shared memory, entries reserved in buf (may run past cap)
    uint32_t cap;
    uint32_t *g_count;
    unsigned long long *g_list;
    uint32_t g_cap;
};

__device__ __forceinline__ void tfe_vs_append(const TfeVsAppender &a, uint32_t vote, bool have, unsigned long long v)
{                                                       // whole warp; vote = ballot of `have`, not zero
    const int lane = threadIdx.x & 31, leader = __ffs(vote) - 1;
    const uint32_t n = __popc(vote), rank = __popc(vote & ((1u << lane) - 1u));
    uint32_t base = 0;
    if (n < 16u) {
        if (lane == leader) base = atomicAdd(a.s_count, n);
        base = __shfl_sync(0xFFFFFFFFu, base, leader);
        if (base + n <= a.cap) {
            if (have) a.buf[base + rank] = v;
            return;
        }
    }
    if (lane == leader) base = atomicAdd(a.g_count, n);
    base = __shfl_sync(0xFFFFFFFFu, base, leader);
    if (have && base + rank < a.g_cap) a.g_list[base + rank] = v;
}

// Whole block; leaves buf cleared and the count at zero.  s_warp: 33 words of shared memory.
__device__ __forceinline__ void tfe_vs_flush(const TfeVsAppender &a, uint32_t *s_warp)
{
    __syncthreads();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t n_s = min(*a.s_count, a.cap);
    __syncthreads();
    for (uint32_t c0 = 0; c0 < n_s; c0 += blockDim.x) {
        const uint32_t i = c0 + threadIdx.x;
        const unsigned long long v = i < n_s ? a.buf[i] : TFE_VS_NONE;
        const bool ok = v != TFE_VS_NONE;
        const uint32_t vote = __ballot_sync(0xFFFFFFFFu, ok);
        if (lane == 0) s_warp[warp] = __popc(vote);
        __syncthreads();
        if (threadIdx.x == 0) {
            uint32_t total = 0;
            for (uint32_t w = 0; w < (blockDim.x >> 5); ++w) { const uint32_t c = s_warp[w]; s_warp[w] = total; total += c; }
            s_warp[32] = total ? atomicAdd(a.g_count, total) : 0u;
        }
        __syncthreads();
        const uint32_t pos = s_warp[32] + s_warp[warp] + __popc(vote & ((1u << lane) - 1u));
        if (ok && pos < a.g_cap) a.g_list[pos] = v;
        __syncthreads();
    }
    for (uint32_t i = threadIdx.x; i < a.cap; i += blockDim.x) a.buf[i] = TFE_VS_NONE;
    if (threadIdx.x == 0) *a.s_count = 0;
    __syncthreads();
}

// A walk over the bookkeeping of the whole table: four quads of slots (128 bytes) per thread and trip; quad g of a
// trip belongs to thread (g mod threads of the grid), so that a stretch of the table is spread over all blocks.
template <bool DECAY>
struct TfeVsTableWalk {
    static constexpr int U = 4;
    const TfeVictimParams &p;
    uint32_t now, n_quads, n_round, stride;
    __device__ __forceinline__ TfeVsTableWalk(const TfeVictimParams &p_, uint32_t now_) : p(p_), now(now_)
    {
        n_quads = (p.C + 3u) >> 2;
        n_round = (n_quads + 31u) & ~31u;              // whole warps stay together
        stride = gridDim.x * blockDim.x;
    }
    // number of slot j of a quad whose bookkeeping is {a, b}
    __device__ __forceinline__ unsigned long long number(const uint4 &a, const uint4 &b, uint32_t quad, int j) const
    {
        const uint2 st = j == 0 ? make_uint2(a.x, a.y) : j == 1 ? make_uint2(a.z, a.w) : j == 2 ? make_uint2(b.x, b.y) : make_uint2(b.z, b.w);
        return ((unsigned long long)tfe_retention_key<DECAY>(st, now, p.div_half_life, p.age_cap) << 32) | (4u * quad + j);
    }
    // f(number, wanted) for the slots of a trip in which some lane of the warp holds a number <= limit (wanted: this
    // one is) -- called by whole warps.  Most trips have none: one vote per sixteen slots, and the numbers are worked
    // out a second time in the trips that have.
    template <class F>
    __device__ __forceinline__ void for_each_up_to(unsigned long long limit, F f) const
    {
        for (uint32_t g = blockIdx.x * blockDim.x + threadIdx.x; g < n_round; g += U * stride) {
            uint4 a[U], b[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const uint32_t gq = g + u * stride;
                a[u] = b[u] = make_uint4(0, 0, 0, 0);
                if (gq < n_quads) {
                    a[u] = __ldcs(reinterpret_cast<const uint4 *>(p.slot_stats) + 2 * (size_t)gq);
                    b[u] = __ldcs(reinterpret_cast<const uint4 *>(p.slot_stats) + 2 * (size_t)gq + 1);
                }
            }
            bool any = false;
#pragma unroll
            for (int u = 0; u < U; ++u)
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const unsigned long long v = number(a[u], b[u], g + u * stride, j);
                    any |= (uint32_t)v < p.C && v <= limit;
                }
            if (!__any_sync(0xFFFFFFFFu, any)) continue;
#pragma unroll
            for (int u = 0; u < U; ++u)
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const unsigned long long v = number(a[u], b[u], g + u * stride, j);
                    f(v, (uint32_t)v < p.C && v <= limit);
                }
        }
    }
};

// f(number, valid) for the first n entries of the candidate list, whole warps together.
template <class F>
__device__ __forceinline__ void tfe_vs_for_each_listed(const unsigned long long *list, uint32_t n, F f)
{
    const uint32_t n_round = (n + 31u) & ~31u;
    for (uint32_t i = blockIdx.x * blockDim.x + threadIdx.x; i < n_round; i += gridDim.x * blockDim.x) {
        const bool in = i < n;
        f(in ? __ldcg(list + i) : 0ull, in);
    }
}

// 64 numbers of a warp, two per lane (v0: position `lane`, v1: position `lane + 32`), sorted ascending by position
// with a bitonic network over shuffles.
__device__ __forceinline__ void tfe_vs_warp_sort64(unsigned long long &v0, unsigned long long &v1, int lane)
{
#pragma unroll
    for (int k = 2; k <= 64; k <<= 1) {
#pragma unroll
        for (int j = k >> 1; j > 0; j >>= 1) {
            if (j == 32) {                               // positions lane and lane + 32 (k = 64: ascending)
                if (v0 > v1) { const unsigned long long t = v0; v0 = v1; v1 = t; }
            } else {
                const unsigned long long o0 = __shfl_xor_sync(0xFFFFFFFFu, v0, j), o1 = __shfl_xor_sync(0xFFFFFFFFu, v1, j);
                const bool lower = (lane & j) == 0;
                const bool up0 = (lane & k) == 0, up1 = ((lane + 32) & k) == 0;
                v0 = (lower == up0) ? (o0 < v0 ? o0 : v0) : (o0 > v0 ? o0 : v0);
                v1 = (lower == up1) ? (o1 < v1 ? o1 : v1) : (o1 > v1 ? o1 : v1);
            }
        }
    }
}

// A number that r or more of the block's 2 * blockDim.x numbers do not exceed (two per thread, all distinct
// except TFE_VS_NONE, of which there are fewer than 2 * blockDim.x - r + 1), and few more than r: every warp
// sorts its 64 and leaves them in `lists`, the first warp then merges the 32 lists up to the r-th smallest.
// s_out: one number.
__device__ __forceinline__ unsigned long long tfe_vs_block_rth(unsigned long long v0, unsigned long long v1, uint32_t r,
                                                                unsigned long long *lists, unsigned long long *s_out)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t n_lists = blockDim.x >> 5;
    // a small r: the r-th smallest of the warps' minima stands in for it.  Those are r distinct numbers of the
    // block, so it is never below the r-th smallest of all, which is all a threshold has to guarantee.
    const bool minima_only = r <= n_lists && r <= 32u;
    uint32_t list_len = 64;
    if (minima_only) {
        const unsigned long long m = v0 < v1 ? v0 : v1;
        const uint32_t m_hi = __reduce_min_sync(0xFFFFFFFFu, (uint32_t)(m >> 32));
        const uint32_t m_lo = __reduce_min_sync(0xFFFFFFFFu, (uint32_t)(m >> 32) == m_hi ? (uint32_t)m : 0xFFFFFFFFu);
        if (lane == 0) lists[warp * 64] = ((unsigned long long)m_hi << 32) | m_lo;
        list_len = 1;
    } else {
        tfe_vs_warp_sort64(v0, v1, lane);
        lists[warp * 64 + lane] = v0;
        lists[warp * 64 + lane + 32] = v1;
    }
    __syncthreads();
    if (warp == 0) {
        uint32_t head = 0;
        unsigned long long cur = (uint32_t)lane < n_lists ? lists[lane * 64] : TFE_VS_NONE;
        unsigned long long picked = TFE_VS_NONE;
        for (uint32_t it = 0; it < r; ++it) {            // r times: the smallest head leaves its list
            const uint32_t m_hi = __reduce_min_sync(0xFFFFFFFFu, (uint32_t)(cur >> 32));
            const uint32_t m_lo = __reduce_min_sync(0xFFFFFFFFu, (uint32_t)(cur >> 32) == m_hi ? (uint32_t)cur : 0xFFFFFFFFu);
            picked = ((unsigned long long)m_hi << 32) | m_lo;
            if (cur == picked && picked != TFE_VS_NONE) {
                ++head;
                cur = head < list_len ? lists[lane * 64 + head] : TFE_VS_NONE;
            }
        }
        if (lane == 0) *s_out = picked;
    }
    __syncthreads();
    return *s_out;
}

template <bool DECAY>
__global__ void __launch_bounds__(TFE_VS_THREADS, 1) tfe_victim_select_kernel(const TfeVictimParams p)
{
    extern __shared__ unsigned long long s_buf[];          // TFE_VS_FINAL_CAP numbers: samples, then collected candidates, then the final set
    __shared__ uint32_t s_hist[TFE_VS_BINS];
    __shared__ uint32_t s_warp[33];
    __shared__ uint32_t s_count;
    __shared__ uint32_t s_pick[4];
    __shared__ uint32_t s_near[TFE_VS_NEAR_BINS];
    __shared__ unsigned long long s_T;
    static_assert(TFE_VS_SAMPLES == 2 * TFE_VS_THREADS, "two samples per thread");
    static_assert(TFE_VS_BINS == 2 * TFE_VS_THREADS, "two pieces of the histogram per thread");
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    TfeVictimState *st = p.st;
    uint32_t boundary = 0;
    tfe_grid_dependency_sync();
    if (*(volatile uint32_t *)&st->status != 0u) return;     // an earlier launch gave up: nothing runs until the host has cleared the state
    const uint32_t now = *p.epoch;
    const TfeVsTableWalk<DECAY> walk(p, now);

    // ---- threshold from a sample, worked out by block 0 for all (148 blocks drawing the same 2,048 slots took
    // 7.5 us, most of it queueing for the same lines of L2): sample i is drawn from the i-th of n_samples equal
    // stretches of the table, so the samples are distinct slots
    unsigned long long T = TFE_VS_NONE;
    if (p.n_samples > 0u && blockIdx.x == 0) {
        unsigned long long v[2];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            // sample number of this thread's h-th value: consecutive stretches of the table go to different warps
            // (a table whose keys all tie is ordered by slot; its smallest samples must not share a warp)
            const uint32_t i = (uint32_t)lane * 64u + 32u * h + (uint32_t)warp;
            v[h] = TFE_VS_NONE;
            if (i < p.n_samples) {
                // stretch i: C / n_samples slots, one more in the first C % n_samples stretches
                const uint32_t len = p.sample_stretch + (i < p.sample_longer ? 1u : 0u);
                const uint32_t s0 = i * p.sample_stretch + min(i, p.sample_longer) +
                                    (uint32_t)tfe_mulhi64(tfe_mix64((unsigned long long)i * 0x9E3779B97F4A7C15ull + 1ull), (unsigned long long)len);
                v[h] = ((unsigned long long)tfe_retention_key<DECAY>(p.slot_stats[s0], now, p.div_half_life, p.age_cap) << 32) | s0;
            }
        }
        T = tfe_vs_block_rth(v[0], v[1], p.sample_rank, s_buf, &s_T);
        if (threadIdx.x == 0) {
            st->threshold = T;
            __threadfence();
            *(volatile uint32_t *)&st->threshold_ready = 1u;
        }
    }
    for (uint32_t i = threadIdx.x; i < TFE_VS_FINAL_CAP; i += blockDim.x) s_buf[i] = TFE_VS_NONE;
    for (uint32_t i = threadIdx.x; i < TFE_VS_NEAR_BINS; i += blockDim.x) s_near[i] = 0;
    if (threadIdx.x == 0) s_count = 0;
    if (p.n_samples > 0u && blockIdx.x != 0) {             // bounded wait for block 0's threshold
        if (threadIdx.x == 0) {
            const volatile uint32_t *ready = &st->threshold_ready, *status = &st->status;
            uint32_t spin = 0;
            while (*ready == 0u && *status == 0u && ++spin <= TFE_SPIN_LIMIT) __nanosleep(40);
            if (*ready == 0u) atomicOr(&st->status, TFE_VS_ERR_BARRIER);
            __threadfence();
            s_T = *(volatile unsigned long long *)&st->threshold;
        }
        __syncthreads();
        T = s_T;
        if (*(volatile uint32_t *)&st->status != 0u) return;
    }
    __syncthreads();

    // ---- scan: candidates (<= T) to the list, smallest and largest number of all
    {
        TfeVsAppender app{s_buf, &s_count, TFE_VS_FINAL_CAP, &st->n_cand, p.list, p.list_cap};
        walk.for_each_up_to(T, [&](unsigned long long v, bool cand) {
            const uint32_t vote = __ballot_sync(0xFFFFFFFFu, cand);
            if (vote == 0u) return;
            tfe_vs_append(app, vote, cand, v);
            if (cand) {                                   // how far below T, on a logarithmic scale
                const uint32_t b = tfe_vs_near_bin(T - v);
                int same;
                __match_all_sync(vote, b, &same);
                if (!same) atomicAdd(&s_near[b], 1u);
                else if (lane == __ffs(vote) - 1) atomicAdd(&s_near[b], (uint32_t)__popc(vote));
            }
        });
        tfe_vs_flush(app, s_warp);                       // synchronises the block
        for (uint32_t i = threadIdx.x; i < TFE_VS_NEAR_BINS; i += blockDim.x)
            if (s_near[i]) atomicAdd(&st->near[i], s_near[i]);
    }
    if (!tfe_vs_boundary(st, boundary)) return;

    // ---- the range [lo, hi] that holds the take-th smallest, `cnt` numbers in it, `k` = its rank inside
    const uint32_t n_cand = __ldcg(&st->n_cand);
    const bool listed = n_cand >= p.take && n_cand <= p.list_cap;      // else: walk the table
    unsigned long long lo = 0ull, hi = 0xFFFFFFFF00000000ull | (p.C - 1u);     // every number lies in [lo, hi]
    uint32_t cnt = p.C, k = p.take;
    if (n_cand >= p.take) {
        // the candidates counted by their distance below T, on a logarithmic scale: the piece that holds the
        // take-th smallest (a few numbers far below the rest do not stretch the range the refine steps divide)
        // (with 128 steps per octave the piece mostly holds few enough numbers to go straight to the final step)
        constexpr int PER = (TFE_VS_NEAR_BINS + TFE_VS_THREADS - 1) / TFE_VS_THREADS;      // consecutive bins per thread
        uint32_t c[PER], mine = 0;
#pragma unroll
        for (int j = 0; j < PER; ++j) {
            const uint32_t i = threadIdx.x * PER + j;
            c[j] = i < TFE_VS_NEAR_BINS ? __ldcg(&st->near[i]) : 0u;
            mine += c[j];
        }
        // numbers beyond this thread's bins (farther below T): a suffix sum over the block
        uint32_t incl = mine;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t u = __shfl_down_sync(0xFFFFFFFFu, incl, o);
            if (lane + o < 32) incl += u;
        }
        if (threadIdx.x == 0) s_pick[0] = 0xFFFFFFFFu;
        if (lane == 0) s_warp[warp] = incl;
        __syncthreads();
        uint32_t beyond = incl - mine;
        for (int w = warp + 1; w < (int)(blockDim.x >> 5); ++w) beyond += s_warp[w];
        if (beyond < p.take && beyond + mine >= p.take) {      // exactly one thread: the take-th smallest is in its bins
            int j = PER - 1;
            for (; j > 0 && beyond + c[j] < p.take; --j) beyond += c[j];
            s_pick[0] = threadIdx.x * PER + j; s_pick[1] = beyond; s_pick[2] = c[j];
        }
        __syncthreads();
        if (s_pick[0] == 0xFFFFFFFFu) {                  // the bins do not add up to n_cand
            if (threadIdx.x == 0) atomicOr(&st->status, TFE_VS_ERR_INTERNAL);
            return;
        }
        unsigned long long d_min, d_max;
        tfe_vs_near_range(s_pick[0], d_min, d_max);
        const unsigned long long piece_lo = T >= d_max ? T - d_max : 0ull, piece_hi = T - d_min;
        lo = piece_lo > lo ? piece_lo : lo;
        hi = piece_hi < hi ? piece_hi : hi;
        k = p.take - s_pick[1];
        cnt = s_pick[2];
        __syncthreads();
    }
    // refine while the set to rank would be large (its cost grows with the square) and the range still splits
    int n_refined = 0;
    for (int it = 0; (p.take - k) + cnt > p.final_cap && cnt > p.range_cap && hi > lo; ++it) {
        if (it >= TFE_VS_MAX_REFINE) {
            if (threadIdx.x == 0) atomicOr(&st->status, TFE_VS_ERR_INTERNAL);
            return;
        }
        n_refined = it + 1;
        const unsigned long long span = hi - lo;
        const int sh = span < (unsigned long long)TFE_VS_BINS ? 0 : (64 - __clzll((long long)span)) - 11;
        for (uint32_t i = threadIdx.x; i < TFE_VS_BINS; i += blockDim.x) s_hist[i] = 0;
        __syncthreads();
        auto count = [&](unsigned long long v, bool valid) {
            if (valid && v >= lo && v <= hi) atomicAdd(&s_hist[(uint32_t)((v - lo) >> sh)], 1u);
        };
        if (listed) tfe_vs_for_each_listed(p.list, n_cand, count);
        else walk.for_each_up_to(hi, count);
        __syncthreads();
        for (uint32_t i = threadIdx.x; i < TFE_VS_BINS; i += blockDim.x)
            if (s_hist[i]) atomicAdd(&st->hist[it][i], s_hist[i]);
        if (!tfe_vs_boundary(st, boundary)) return;
        // the piece that holds the k-th smallest of the range: every block works it out for itself
        {
            const uint32_t h0 = __ldcg(&st->hist[it][2 * threadIdx.x]), h1 = __ldcg(&st->hist[it][2 * threadIdx.x + 1]);
            const uint32_t sum = h0 + h1;
            uint32_t incl = sum;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const uint32_t u = __shfl_up_sync(0xFFFFFFFFu, incl, o);
                if (lane >= o) incl += u;
            }
            if (threadIdx.x == 0) s_pick[0] = 0xFFFFFFFFu;
            if (lane == 31) s_warp[warp] = incl;
            __syncthreads();
            for (int w = 0; w < warp; ++w) incl += s_warp[w];
            if (incl >= k && incl - sum < k) {           // exactly one thread
                const uint32_t before = incl - sum;
                const bool second = k - before > h0;
                s_pick[0] = 2 * threadIdx.x + (second ? 1u : 0u);
                s_pick[1] = before + (second ? h0 : 0u);
                s_pick[2] = second ? h1 : h0;
            }
            __syncthreads();
            if (s_pick[0] == 0xFFFFFFFFu) {              // the histogram holds fewer than k numbers
                if (threadIdx.x == 0) atomicOr(&st->status, TFE_VS_ERR_INTERNAL);
                return;
            }
            const unsigned long long piece_lo = lo + ((unsigned long long)s_pick[0] << sh);
            const unsigned long long piece_hi = piece_lo + ((1ull << sh) - 1ull);
            lo = piece_lo;
            hi = piece_hi < hi ? piece_hi : hi;
            k -= s_pick[1];
            cnt = s_pick[2];
            __syncthreads();
        }
    }

    // ---- final: gather everything <= hi, rank it
    {
        TfeVsAppender app{s_buf, &s_count, TFE_VS_FINAL_CAP, &st->n_final, p.fin, (uint32_t)TFE_VS_FINAL_CAP};
        auto gather = [&](unsigned long long v, bool valid) {
            const bool have = valid && v <= hi;
            const uint32_t vote = __ballot_sync(0xFFFFFFFFu, have);
            if (vote) tfe_vs_append(app, vote, have, v);
        };
        if (listed) tfe_vs_for_each_listed(p.list, n_cand, gather);
        else walk.for_each_up_to(hi, gather);
        tfe_vs_flush(app, s_warp);
    }
    if (!tfe_vs_boundary(st, boundary)) return;
    const uint32_t n_final = __ldcg(&st->n_final);
    if (n_final != (p.take - k) + cnt || n_final > (uint32_t)TFE_VS_FINAL_CAP) {
        if (threadIdx.x == 0) atomicOr(&st->status, TFE_VS_ERR_INTERNAL);
        return;
    }
    for (uint32_t i = threadIdx.x; i < n_final; i += blockDim.x) s_buf[i] = __ldcg(p.fin + i);
    __syncthreads();
    // one number per warp and trip, dealt to the blocks first so that a small set still uses every SM
    for (uint32_t e = warp * gridDim.x + blockIdx.x; e < n_final; e += gridDim.x * (blockDim.x >> 5)) {
        const unsigned long long x = s_buf[e];
        uint32_t below = 0;
#pragma unroll 8
        for (uint32_t i = lane; i < n_final; i += 32) below += s_buf[i] < x;
        below = __reduce_add_sync(0xFFFFFFFFu, below);
        if (lane == 0 && below < p.take) {
            p.out_slots[below] = (int32_t)(uint32_t)x;
            p.out_keys[below] = (uint32_t)(x >> 32);
        }
    }
    // ---- ready for the next launch: every block is past its last read of the counts by distance and of the
    // histograms (they were read before the boundary above); the counters go when the last block leaves
    for (uint32_t i = blockIdx.x * blockDim.x + threadIdx.x; i < TFE_VS_NEAR_BINS; i += gridDim.x * blockDim.x) st->near[i] = 0u;
    for (uint32_t i = blockIdx.x * blockDim.x + threadIdx.x; i < (uint32_t)n_refined * TFE_VS_BINS; i += gridDim.x * blockDim.x)
        (&st->hist[0][0])[i] = 0u;
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        if (atomicAdd(&st->left, 1u) == gridDim.x - 1u) {
            st->arrived = 0u; st->n_cand = 0u; st->n_final = 0u; st->threshold_ready = 0u; st->left = 0u;
        }
    }
}


// ------------------------------------------------ index construction on the device
//
// The cold step of the method (the paper's index construction is its dominant offline cost):
// N phrases -> keys -> two-choice cuckoo placement in buckets of four 16-byte slots, all on the
// GPU.  A slot {key, value} is written and moved with 128-bit atomics, so every slot always holds
// one whole entry and the placement needs no locks:
//
//   tfe_build_insert_kernel   one thread per phrase: checks its length, ids and residency, forms
//                             the key, claims its GPU-tier slot in the owner array, then
//                             compare-and-swaps the entry into a free slot of either bucket; if
//                             both are full it exchanges with a resident entry and carries that
//                             one to its other bucket (bounded number of moves)
//   tfe_build_verify_kernel   one thread per phrase: looks its own key up and records where it
//                             sits; finding another phrase under the key means two phrases share
//                             it -- the same tuple twice, or (hashed orders) two tuples, one hash
// Problems are reported as bits of a status word; the host turns them into error codes.
#define TFE_BUILD_BAD_PHRASE 1u         // length not a configured order, id outside the vocabulary, residency < -2
#define TFE_BUILD_BAD_SLOT 2u           // GPU-tier slot out of range or claimed twice
#define TFE_BUILD_KICKS 4u              // an insertion ran out of moves
#define TFE_BUILD_DUPLICATE 8u
#define TFE_BUILD_COLLISION 16u
#define TFE_BUILD_LOST 32u              // a phrase is not where a lookup would find it

__device__ __forceinline__ ulonglong2 atomic_cas_slot(ulonglong2 *slot, ulonglong2 expect, ulonglong2 put)
{
    ulonglong2 old;
    asm volatile(
        "{\n\t.reg .b128 o, n, c;\n\t"
        "mov.b128 c, {%2, %3};\n\t"
        "mov.b128 n, {%4, %5};\n\t"
        "atom.global.cas.b128 o, [%6], c, n;\n\t"
        "mov.b128 {%0, %1}, o;\n\t}"
        : "=l"(old.x), "=l"(old.y)
        : "l"(expect.x), "l"(expect.y), "l"(put.x), "l"(put.y), "l"(slot)
        : "memory");
    return old;
}

__device__ __forceinline__ ulonglong2 atomic_exch_slot(ulonglong2 *slot, ulonglong2 put)
{
    ulonglong2 old;
    asm volatile(
        "{\n\t.reg .b128 o, n;\n\t"
        "mov.b128 n, {%2, %3};\n\t"
        "atom.global.exch.b128 o, [%4], n;\n\t"
        "mov.b128 {%0, %1}, o;\n\t}"
        : "=l"(old.x), "=l"(old.y)
        : "l"(put.x), "l"(put.y), "l"(slot)
        : "memory");
    return old;
}

struct TfeBuildParams {
    const int4 *phrase_tokens;      // [N]
    const uint8_t *phrase_len;      // [N]
    const int32_t *init_slot;       // [N]
    uint32_t n_phrases;
    int64_t gpu_slots;
    int32_t vocab, tok_bits;
    uint32_t order_mask;            // bit n set: n is a configured order
    uint32_t hashed_mask;           // bit n set: order n is hashed
    int32_t max_kicks;
    ulonglong2 *index;
    uint64_t n_buckets;
    uint32_t *slot_owner;           // [C], preset to "no owner"
    uint32_t *phrase_pos;           // [N]
    uint32_t *status;
};

// Key of phrase i, or 0 if its length is not a configured order or it holds an id outside the vocabulary.
__device__ __forceinline__ unsigned long long tfe_build_key(const TfeBuildParams &p, uint32_t i)
{
    const int n = p.phrase_len[i];
    if (n < 1 || n > 4 || !((p.order_mask >> n) & 1u)) return 0ull;
    const int4 t = p.phrase_tokens[i];
    const int32_t tok[4] = {t.x, t.y, t.z, t.w};
    int32_t tk[4] = {-1, -1, -1, -1};       // tk[j] = id at distance j before the phrase's last token
    bool ok = true;
#pragma unroll
    for (int j = 0; j < 4; ++j)
        if (j < n) {
            const int32_t x = tok[n - 1 - j];
            if (x < 0 || x >= p.vocab) ok = false;
            tk[j] = x;
        }
    return ok ? tfe_make_key(n, tk, p.tok_bits) : 0ull;
}

__global__ void __launch_bounds__(256)
tfe_build_insert_kernel(const TfeBuildParams p)
{
    const uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= p.n_phrases) return;
    ulonglong2 cur;
    cur.x = tfe_build_key(p, i);
    const int32_t res = p.init_slot[i];
    if (cur.x == 0ull || res < -2) {
        atomicOr(p.status, TFE_BUILD_BAD_PHRASE);
        return;
    }
    if (res >= 0) {
        if ((int64_t)res >= p.gpu_slots || atomicCAS(&p.slot_owner[res], 0xFFFFFFFFu, i) != 0xFFFFFFFFu) {
            atomicOr(p.status, TFE_BUILD_BAD_SLOT);
            return;
        }
    }
    cur.y = ((unsigned long long)i << 32) | (uint32_t)res;
    const ulonglong2 empty = make_ulonglong2(0ull, 0ull);
    uint64_t first = tfe_home_bucket_of(cur.x, p.n_buckets);
    uint32_t rng = i * 2654435761u + 12345u;
    for (int32_t kick = 0; kick <= p.max_kicks; ++kick) {
        // a free slot in the bucket at hand, then in the entry's other bucket
        const uint64_t home = tfe_home_bucket_of(cur.x, p.n_buckets);
        const uint64_t second = tfe_second_bucket_of(cur.x, home, p.n_buckets);
        const uint64_t other = first == home ? second : home;
#pragma unroll
        for (int which = 0; which < 2; ++which) {
            ulonglong2 *bucket = p.index + (which == 0 ? first : other) * TFE_SLOTS_PER_BUCKET;
            for (int sl = 0; sl < TFE_SLOTS_PER_BUCKET; ++sl) {
                if (__ldcg(&bucket[sl].x) != 0ull) continue;
                if (atomic_cas_slot(bucket + sl, empty, cur).x == 0ull) return;      // placed
            }
        }
        // both full: take the place of a resident entry of the bucket at hand and carry that one
        // to its other bucket (the walk moves on from there)
        rng = rng * 1664525u + 1013904223u;
        ulonglong2 *victim = p.index + first * TFE_SLOTS_PER_BUCKET + (rng >> 30);
        const ulonglong2 out = atomic_exch_slot(victim, cur);
        if (out.x == 0ull) return;          // cannot happen (slots are never emptied); placed either way
        cur = out;
        const uint64_t h2 = tfe_home_bucket_of(cur.x, p.n_buckets);
        first = h2 == first ? tfe_second_bucket_of(cur.x, h2, p.n_buckets) : h2;
    }
    atomicOr(p.status, TFE_BUILD_KICKS);
}

__global__ void __launch_bounds__(256)
tfe_build_verify_kernel(const TfeBuildParams p)
{
    const uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= p.n_phrases) return;
    const unsigned long long key = tfe_build_key(p, i);
    if (key == 0ull) return;
    const uint64_t b1 = tfe_home_bucket_of(key, p.n_buckets);
    const uint64_t b2 = tfe_second_bucket_of(key, b1, p.n_buckets);
    uint32_t found = 0xFFFFFFFFu, mine = 0xFFFFFFFFu;
#pragma unroll
    for (int which = 0; which < 2; ++which) {
        const uint64_t b = which == 0 ? b1 : b2;
        const ulonglong2 *bucket = p.index + b * TFE_SLOTS_PER_BUCKET;
        for (int sl = 0; sl < TFE_SLOTS_PER_BUCKET; ++sl) {
            const ulonglong2 e = bucket[sl];
            if (e.x != key) continue;
            const uint32_t id = (uint32_t)(e.y >> 32);
            if (id == i) mine = (uint32_t)(b * TFE_SLOTS_PER_BUCKET + sl); else found = id;
        }
        if (b2 == b1) break;
    }
    if (mine == 0xFFFFFFFFu) atomicOr(p.status, TFE_BUILD_LOST);
    else p.phrase_pos[i] = mine;            // where the entry sits (the install kernel rewrites its value there)
    if (found != 0xFFFFFFFFu) {
        const int n = p.phrase_len[i];
        bool same = p.phrase_len[found] == n;
        if (same && ((p.hashed_mask >> n) & 1u)) {
            const int4 a = p.phrase_tokens[i], b = p.phrase_tokens[found];
            const int32_t ta[4] = {a.x, a.y, a.z, a.w}, tb[4] = {b.x, b.y, b.z, b.w};
            for (int j = 0; j < n; ++j) same = same && ta[j] == tb[j];
        }
        atomicOr(p.status, same ? TFE_BUILD_DUPLICATE : TFE_BUILD_COLLISION);
    }
}

// Residency of every phrase as the index holds it (>= 0 slot, -1 host, -2 SSD): the host-side
// mirror of a context built on the device is filled from this on its first use.
__global__ void __launch_bounds__(256)
tfe_gather_residency_kernel(const ulonglong2 *index, const uint32_t *phrase_pos, uint32_t n_phrases, int32_t *out)
{
    const uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n_phrases) out[i] = (int32_t)(uint32_t)index[phrase_pos[i]].y;
}
