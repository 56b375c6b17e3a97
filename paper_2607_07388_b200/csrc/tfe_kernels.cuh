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
#define TFE_MIN_BLOCKS_GENERAL 2     // blocks per SM the COSINE variants are compiled for (the others: TFE_MIN_BLOCKS)
#endif
#ifndef TFE_MIN_BLOCKS
#define TFE_MIN_BLOCKS 3
#endif

template <int HT, bool ALL, bool COS, bool PACKED>
__global__ void __launch_bounds__(TFE_BLOCK_THREADS, COS ? TFE_MIN_BLOCKS_GENERAL : TFE_MIN_BLOCKS)
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
template <int HT, bool PACKED, bool RANGED, int UNROLL>
__global__ void __launch_bounds__(TFE_BLOCK_THREADS, UNROLL == 4 ? TFE_MIN_BLOCKS : TFE_MIN_BLOCKS + 1)
tfe_lookup_inject_longest_kernel(const TfeLookupParams p)
{
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
                        for (int e = 0; e < VN; ++e) y[e] = fmaf(p.lambda, m[e], x[e]);
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
//   tfe_install_claim_kernel<0>  every entry stamps its phrase
//   tfe_install_claim_kernel<1>  every candidate stamps its slot
//   tfe_install_device_kernel    one warp per entry: the winners install (as tfe_install_kernel)
//   tfe_install_clear_kernel     the stamps this call wrote go back to zero
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
    uint32_t *count;                // entries applied (cleared by the host side before the launches)
    uint2 *slot_stats;
    const uint32_t *epoch;
};

__device__ __forceinline__ bool tfe_install_candidate(const TfeInstallDeviceParams &p, int k)
{
    const uint32_t id = p.ids[k];
    const int32_t dst = p.dst_slots[k];
    if (id >= p.n_phrases || dst < 0 || (int64_t)dst >= p.gpu_slots) return false;
    if ((int32_t)(uint32_t)p.index[p.phrase_pos[id]].y >= 0) return false;          // resident before the call
    return __ldcg(p.phrase_stamp + id) == (uint32_t)(TFE_INSTALL_DEVICE_MAX - k);
}

template <int STAGE>
__global__ void __launch_bounds__(256)
tfe_install_claim_kernel(const TfeInstallDeviceParams p)
{
    tfe_grid_dependency_sync();
    const int k = blockIdx.x * blockDim.x + threadIdx.x;
    if (k >= p.n) return;
    const uint32_t stamp = (uint32_t)(TFE_INSTALL_DEVICE_MAX - k);         // 1..4096: never the cleared value
    if (STAGE == 0) {
        const uint32_t id = p.ids[k];
        if (id < p.n_phrases) atomicMax(p.phrase_stamp + id, stamp);
    } else {
        if (tfe_install_candidate(p, k)) atomicMax(p.slot_stamp + p.dst_slots[k], stamp);
    }
}

__global__ void __launch_bounds__(256)
tfe_install_clear_kernel(const TfeInstallDeviceParams p)
{
    tfe_grid_dependency_sync();
    const int k = blockIdx.x * blockDim.x + threadIdx.x;
    if (k >= p.n) return;
    const uint32_t id = p.ids[k];
    const int32_t dst = p.dst_slots[k];
    if (id < p.n_phrases) p.phrase_stamp[id] = 0;
    if (dst >= 0 && (int64_t)dst < p.gpu_slots) p.slot_stamp[dst] = 0;
}

__global__ void __launch_bounds__(TFE_BLOCK_THREADS)
tfe_install_device_kernel(const TfeInstallDeviceParams p)
{
    tfe_grid_dependency_sync();
    const int lane = threadIdx.x & 31;
    const int k = blockIdx.x * TFE_WARPS_PER_BLOCK + (threadIdx.x >> 5);
    if (k >= p.n) return;
    bool apply = false;
    if (lane == 0) {
        apply = tfe_install_candidate(p, k) &&
                __ldcg(p.slot_stamp + p.dst_slots[k]) == (uint32_t)(TFE_INSTALL_DEVICE_MAX - k);
        if (p.applied) p.applied[k] = apply ? 1 : 0;
        if (apply) atomicAdd(p.count, 1u);
    }
    apply = __shfl_sync(0xFFFFFFFFu, apply, 0);
    if (!apply) return;
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
// 64-bit number per slot, so this is a selection of the n smallest of C distinct numbers:
//
//   tfe_victim_pass_kernel   x3 over the key's 32 bits, most significant digit first (11,11,10 bits):
//                            histogram of the digit over the slots that agree with the digits chosen so
//                            far; the block that finishes last picks the digit holding the n-th smallest
//                            and re-arms the histogram.  The first pass computes and stores the keys.
//   tfe_victim_tie_kernel    the slot half of the n-th smallest: a count of the slots that hold exactly
//                            its key, in slot (= memory) order, instead of three more digit passes
//   tfe_victim_collect_kernel  appends every number <= the n-th smallest to a list (any order)
//   tfe_victim_sort_kernel     one block: bitonic sort of the list, writes slots and keys
#define TFE_VICTIMS_MAX 4096
#define TFE_VICTIM_BINS 2048

struct TfeVictimState {
    unsigned long long prefix;      // digits chosen so far, in place
    uint32_t k_rem;                 // rank (1-based) of the wanted number among those sharing the prefix
    uint32_t ticket;                // blocks done in the current pass
    uint32_t n_out;                 // entries appended by the collect kernel
    uint32_t pad;
};

__device__ __forceinline__ uint32_t tfe_retention_key(uint2 st, uint32_t owner, uint32_t now, int32_t half_life)
{
    if (owner == 0xFFFFFFFFu) return 0u;
    const uint32_t age = now - st.y;
    const uint32_t shift = half_life > 0 ? min(31u, age / (uint32_t)half_life) : 0u;
    return (min(st.x >> shift, 65535u) << 16) | (65535u - min(age, 65535u));
}

#define TFE_VICTIM_THREADS 512

// slot_stats, slot_owner and slot_key hold a multiple of 4 entries (the tail is padding).
template <bool FIRST>
__global__ void __launch_bounds__(TFE_VICTIM_THREADS)
tfe_victim_pass_kernel(const uint2 *slot_stats, const uint32_t *slot_owner, const uint32_t *epoch, int32_t half_life,
                       uint32_t *slot_key, uint32_t C, uint32_t n_first, int shift, int bits, uint32_t *hist,
                       TfeVictimState *state)
{
    __shared__ uint32_t s_hist[TFE_VICTIM_BINS];
    __shared__ uint32_t s_part[256];
    __shared__ uint32_t s_last;
    for (int i = threadIdx.x; i < TFE_VICTIM_BINS; i += blockDim.x) s_hist[i] = 0;
    __syncthreads();
    tfe_grid_dependency_sync();                 // the pass before this one decides the prefix
    const unsigned long long prefix = FIRST ? 0ull : state->prefix;
    const uint32_t now = FIRST ? *epoch : 0u;
    const int above = shift + bits;             // bits above this digit are decided
    const uint32_t mask = (1u << bits) - 1u;
    const uint32_t n_quads = (C + 3u) >> 2;
    const uint32_t n_round = (n_quads + 31u) & ~31u;    // whole warps stay together for the match
    const uint32_t stride = gridDim.x * blockDim.x;
    uint32_t g = blockIdx.x * blockDim.x + threadIdx.x;
    uint4 nxt = make_uint4(0, 0, 0, 0);         // the keys one iteration ahead (later passes)
    if (!FIRST && g < n_quads) nxt = reinterpret_cast<const uint4 *>(slot_key)[g];
    for (; g < n_round; g += stride) {
        uint32_t key[4] = {0, 0, 0, 0};
        if (FIRST) {
            if (g < n_quads) {
                const uint4 a = __ldcs(reinterpret_cast<const uint4 *>(slot_stats) + 2 * g);
                const uint4 b = __ldcs(reinterpret_cast<const uint4 *>(slot_stats) + 2 * g + 1);
                const uint4 o = __ldcs(reinterpret_cast<const uint4 *>(slot_owner) + g);
                key[0] = tfe_retention_key(make_uint2(a.x, a.y), o.x, now, half_life);
                key[1] = tfe_retention_key(make_uint2(a.z, a.w), o.y, now, half_life);
                key[2] = tfe_retention_key(make_uint2(b.x, b.y), o.z, now, half_life);
                key[3] = tfe_retention_key(make_uint2(b.z, b.w), o.w, now, half_life);
                reinterpret_cast<uint4 *>(slot_key)[g] = make_uint4(key[0], key[1], key[2], key[3]);
            }
        } else {
            key[0] = nxt.x; key[1] = nxt.y; key[2] = nxt.z; key[3] = nxt.w;
            if (g + stride < n_quads) nxt = reinterpret_cast<const uint4 *>(slot_key)[g + stride];
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const uint32_t s0 = 4 * g + j;
            const unsigned long long comp = ((unsigned long long)key[j] << 32) | s0;
            const bool live = s0 < C && g < n_quads && (above >= 64 || (comp >> above) == (prefix >> above));
            const uint32_t digit = (uint32_t)(comp >> shift) & mask;
            // one shared-memory atomic per distinct digit of the warp
            const uint32_t vote = __ballot_sync(0xFFFFFFFFu, live);
            if (live) {
                const uint32_t peers = __match_any_sync(vote, digit);
                if ((threadIdx.x & 31) == __ffs(peers) - 1) atomicAdd(&s_hist[digit], __popc(peers));
            }
        }
    }
    __syncthreads();
    for (int i = threadIdx.x; i < TFE_VICTIM_BINS; i += blockDim.x)
        if (s_hist[i]) atomicAdd(&hist[i], s_hist[i]);
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) s_last = atomicAdd(&state->ticket, 1u) == gridDim.x - 1;
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    // ---- last block: the digit whose bin holds the k_rem-th smallest
    constexpr int PER = TFE_VICTIM_BINS / 256;
    uint32_t mine[PER], sum = 0;
    if (threadIdx.x < 256) {
#pragma unroll
        for (int j = 0; j < PER; ++j) {
            mine[j] = __ldcg(hist + threadIdx.x * PER + j);
            hist[threadIdx.x * PER + j] = 0;
            sum += mine[j];
        }
        s_part[threadIdx.x] = sum;
    }
    __syncthreads();
    // inclusive scan of the 256 partial sums by the first 8 warps, then the thread whose range
    // holds the k-th smallest announces itself
    const uint32_t k_want = FIRST ? n_first : state->k_rem;
    uint32_t incl = 0;
    if (threadIdx.x < 256) {
        incl = sum;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t v = __shfl_up_sync(0xFFFFFFFFu, incl, o);
            if ((threadIdx.x & 31) >= o) incl += v;
        }
        if ((threadIdx.x & 31) == 31) s_hist[threadIdx.x >> 5] = incl;      // warp totals
    }
    __syncthreads();
    if (threadIdx.x < 256) {
        for (int wq = 0; wq < (int)(threadIdx.x >> 5); ++wq) incl += s_hist[wq];
        if (incl >= k_want && incl - sum < k_want) {
            s_part[0] = threadIdx.x;                // owning thread (exactly one)
            s_hist[8] = k_want - (incl - sum);      // rank within its bins
        }
    }
    __syncthreads();
    if (threadIdx.x < 256 && threadIdx.x == s_part[0]) {
        uint32_t k = s_hist[8];
        int j = 0;
        for (; j < PER - 1 && mine[j] < k; ++j) k -= mine[j];
        state->prefix = prefix | ((unsigned long long)(threadIdx.x * PER + j) << shift);
        state->k_rem = k;
        state->ticket = 0;
    }
}

// After the three passes over the key's 32 bits the wanted number is known to be the k_rem-th smallest
// SLOT among those holding exactly that key.  Slot order is memory order, so no further digit passes are
// needed: every block counts the ties of one contiguous range of slots; the block that finishes last
// scans the per-block counts, finds the range that holds the k_rem-th tie, walks that range once more and
// completes state->prefix with the slot.  `tie_count` is the (zeroed) histogram array, left zeroed again.
__global__ void __launch_bounds__(TFE_VICTIM_THREADS)
tfe_victim_tie_kernel(const uint32_t *slot_key, uint32_t C, uint32_t *tie_count, TfeVictimState *state)
{
    __shared__ uint32_t s_warp[TFE_VICTIM_THREADS / 32];
    __shared__ uint32_t s_last, s_block, s_rank;
    tfe_grid_dependency_sync();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const unsigned long long prefix = state->prefix;
    const uint32_t key_star = (uint32_t)(prefix >> 32);
    const uint32_t n_quads = (C + 3u) >> 2;
    const uint32_t per_block = (n_quads + gridDim.x - 1) / gridDim.x;
    auto ties_of = [&](uint32_t g) -> uint32_t {            // slots of quad g that hold the key
        const uint4 k4 = __ldcg(reinterpret_cast<const uint4 *>(slot_key) + g);
        return (uint32_t)(k4.x == key_star && 4 * g < C) + (uint32_t)(k4.y == key_star && 4 * g + 1 < C) +
               (uint32_t)(k4.z == key_star && 4 * g + 2 < C) + (uint32_t)(k4.w == key_star && 4 * g + 3 < C);
    };
    {
        const uint32_t q0 = min(n_quads, blockIdx.x * per_block), q1 = min(n_quads, q0 + per_block);
        uint32_t mine = 0;
        for (uint32_t g = q0 + threadIdx.x; g < q1; g += blockDim.x) mine += ties_of(g);
        mine = __reduce_add_sync(0xFFFFFFFFu, mine);
        if (lane == 0) s_warp[warp] = mine;
        __syncthreads();
        if (threadIdx.x == 0) {
            uint32_t total = 0;
            for (int w = 0; w < TFE_VICTIM_THREADS / 32; ++w) total += s_warp[w];
            tie_count[blockIdx.x] = total;
            __threadfence();
            s_last = atomicAdd(&state->ticket, 1u) == gridDim.x - 1;
        }
        __syncthreads();
        if (!s_last) return;
        __threadfence();
    }
    // ---- last block: which range holds the k_rem-th tie.  The per-block counts (at most two per thread,
    // loaded together) are scanned in block order: first all threads' first element, then the second ones.
    {
        const uint32_t want = state->k_rem;
        uint32_t c[2], incl[2];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const uint32_t i = h * TFE_VICTIM_THREADS + threadIdx.x;
            c[h] = i < gridDim.x ? __ldcg(tie_count + i) : 0u;
            if (i < gridDim.x) tie_count[i] = 0;
        }
        uint32_t carry = 0;                                   // total of the first half, for the second
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            uint32_t v = c[h];
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const uint32_t u = __shfl_up_sync(0xFFFFFFFFu, v, o);
                if (lane >= o) v += u;
            }
            __syncthreads();
            if (lane == 31) s_warp[warp] = v;
            __syncthreads();
            uint32_t before = carry, total = 0;
            for (int w = 0; w < TFE_VICTIM_THREADS / 32; ++w) {
                if (w < warp) before += s_warp[w];
                total += s_warp[w];
            }
            incl[h] = before + v;
            carry += total;
        }
        if (threadIdx.x == 0) { s_block = 0; s_rank = 0; }      // overwritten below: k_rem <= number of ties
        __syncthreads();
#pragma unroll
        for (int h = 0; h < 2; ++h)
            if (incl[h] >= want && incl[h] - c[h] < want) {      // exactly one element
                s_block = h * TFE_VICTIM_THREADS + threadIdx.x;
                s_rank = want - (incl[h] - c[h]);
            }
    }
    __syncthreads();
    // ---- walk that range: a contiguous piece per thread, counts, scan, then the piece that holds the tie
    const uint32_t q0 = min(n_quads, s_block * per_block), q1 = min(n_quads, q0 + per_block);
    const uint32_t per_thread = (q1 - q0 + blockDim.x - 1) / blockDim.x;
    const uint32_t t0 = min(q1, q0 + threadIdx.x * per_thread), t1 = min(q1, t0 + per_thread);
    uint32_t mine = 0;
    for (uint32_t g = t0; g < t1; ++g) mine += ties_of(g);
    uint32_t incl = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t v = __shfl_up_sync(0xFFFFFFFFu, incl, o);
        if (lane >= o) incl += v;
    }
    __syncthreads();
    if (lane == 31) s_warp[warp] = incl;
    __syncthreads();
    uint32_t before = incl - mine;
    for (int w = 0; w < warp; ++w) before += s_warp[w];
    const uint32_t want = s_rank;
    if (want > before && want <= before + mine) {          // exactly one thread
        uint32_t left = want - before;
        for (uint32_t g = t0; g < t1 && left; ++g) {
            const uint4 k4 = __ldcg(reinterpret_cast<const uint4 *>(slot_key) + g);
            const uint32_t key[4] = {k4.x, k4.y, k4.z, k4.w};
#pragma unroll
            for (int j = 0; j < 4; ++j)
                if (left && key[j] == key_star && 4 * g + j < C && --left == 0)
                    state->prefix = (prefix & 0xFFFFFFFF00000000ull) | (4 * g + j);
        }
    }
    if (threadIdx.x == 0) state->ticket = 0;
}

__global__ void __launch_bounds__(TFE_VICTIM_THREADS)
tfe_victim_collect_kernel(const uint32_t *slot_key, uint32_t C, TfeVictimState *state, unsigned long long *list,
                          uint32_t cap)
{
    tfe_grid_dependency_sync();
    const unsigned long long limit = state->prefix;
    const uint32_t n_quads = (C + 3u) >> 2;
    for (uint32_t g = blockIdx.x * blockDim.x + threadIdx.x; g < n_quads; g += gridDim.x * blockDim.x) {
        const uint4 k4 = reinterpret_cast<const uint4 *>(slot_key)[g];
        const uint32_t key[4] = {k4.x, k4.y, k4.z, k4.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const uint32_t s0 = 4 * g + j;
            const unsigned long long comp = ((unsigned long long)key[j] << 32) | s0;
            if (s0 < C && comp <= limit) {
                const uint32_t at = atomicAdd(&state->n_out, 1u);
                if (at < cap) list[at] = comp;
            }
        }
    }
}

// One block sorts the selected composites (at most TFE_VICTIMS_MAX = 4,096) ascending: a bitonic network
// with four consecutive elements per thread.  Compare-exchange distances 1 and 2 stay inside a thread,
// distances 4..64 are warp shuffles, only distances >= 128 go through shared memory (15 of the 78 steps at
// 4,096 elements).
__global__ void __launch_bounds__(1024)
tfe_victim_sort_kernel(const unsigned long long *list, TfeVictimState *state, uint32_t n, int32_t *out_slots,
                       uint32_t *out_keys)
{
    static_assert(TFE_VICTIMS_MAX == 4 * 1024, "four elements per thread of a 1,024-thread block");
    __shared__ unsigned long long s_v[TFE_VICTIMS_MAX];
    uint32_t pow2 = 1;
    while (pow2 < n) pow2 <<= 1;
    tfe_grid_dependency_sync();
    const uint32_t base = 4u * threadIdx.x;
    unsigned long long v[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) v[e] = base + e < n ? list[base + e] : ~0ull;      // padding sorts to the end
    for (uint32_t k = 2; k <= pow2; k <<= 1) {
        uint32_t j = k >> 1;
        if (j >= 128) {
#pragma unroll
            for (int e = 0; e < 4; ++e) s_v[base + e] = v[e];
            __syncthreads();
            for (; j >= 128; j >>= 1) {
                for (uint32_t t = threadIdx.x; t < TFE_VICTIMS_MAX / 2; t += blockDim.x) {
                    const uint32_t i = ((t & ~(j - 1)) << 1) | (t & (j - 1));      // the pair's lower index
                    const uint32_t l = i | j;
                    const unsigned long long a = s_v[i], b = s_v[l];
                    const bool up = (i & k) == 0;
                    if ((a > b) == up) { s_v[i] = b; s_v[l] = a; }
                }
                __syncthreads();
            }
#pragma unroll
            for (int e = 0; e < 4; ++e) v[e] = s_v[base + e];
        }
        for (; j >= 4; j >>= 1) {                   // partner element in another lane of this warp
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const unsigned long long other = __shfl_xor_sync(0xFFFFFFFFu, v[e], (int)(j >> 2));
                const uint32_t i = base + e;
                const bool up = (i & k) == 0, lower = (i & j) == 0;
                v[e] = (lower == up) ? (other < v[e] ? other : v[e]) : (other > v[e] ? other : v[e]);
            }
        }
        // partner element in this thread: distance 2 (from k = 4 on), then distance 1
        auto exchange = [&](unsigned long long &a, unsigned long long &b, uint32_t i) {
            const bool up = (i & k) == 0;
            if ((a > b) == up) { const unsigned long long t = a; a = b; b = t; }
        };
        if (k >= 4) { exchange(v[0], v[2], base); exchange(v[1], v[3], base + 1); }
        exchange(v[0], v[1], base);
        exchange(v[2], v[3], base + 2);
    }
#pragma unroll
    for (int e = 0; e < 4; ++e)
        if (base + e < n) {
            out_slots[base + e] = (int32_t)(uint32_t)v[e];
            out_keys[base + e] = (uint32_t)(v[e] >> 32);
        }
    if (threadIdx.x == 0) state->n_out = 0;      // re-armed for the next selection
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
