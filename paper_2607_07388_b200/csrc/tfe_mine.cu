// N-gram extraction with a frequency threshold (paper Sec. 4.2, construction pipeline: candidate phrases
// such as bigrams and trigrams selected by a frequency threshold; Sec. 5.3: this tokenizer-level n-gram
// extraction is the dominant offline cost of building a table).
//
// Input: a tokenised corpus on the device, int32 [L]; an id outside [0, vocab) separates documents.  For
// every configured order n and end position t whose n ids are valid, the tuple x_{t-n+1..t} occurs once.
// Output: every tuple that occurs at least min_count times, with its count, in ascending (end position of
// its first occurrence, n) order -- the phrase table that tfe_index_build_device takes.
//
// No sort: counting is a hash-table pass, the order comes from the corpus itself.
//
//   tfe_mine_count_kernel   two end positions per thread.  The window's exact 64-bit key (ids packed side
//                           by side; an order too wide for 64 bits is keyed by the table slots of its two
//                           halves, which are exact names of those bigrams) is inserted into an
//                           open-addressing table of 16-byte slots {key, count, first} by a 64-bit
//                           compare-and-swap on the key; equal keys are combined first inside a warp
//                           (match.any) and inside the block (shared-memory table), then one atomicAdd on
//                           the count and, only where it can lower it, one atomicMin on the first end
//                           position.
//   tfe_mine_mark_kernel    one sequential sweep over the table: every occupied slot is one distinct tuple --
//                           counted, added to the histogram of counts and, if the count reaches the
//                           threshold, scattered as val[first] = count into the per-position array (0
//                           everywhere else).  The table is then reused by the next order.
//   tfe_mine_block_sums / tfe_mine_scan / tfe_mine_emit
//                           ordered compaction over (position, order): per-block totals, their exclusive
//                           scan, and the writes of tuple, length and count at the scanned offsets.
//
// All loops over table slots are bounded by the table's size; a probe that runs out sets an error word.
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdint>
#include <cstring>
#include <vector>

#include "../../include/tfe.h"

namespace {

constexpr int kThreads = 256;
constexpr int kPosPerThread = 4;                       // emit / block-sum kernels
constexpr int kPosPerBlock = kThreads * kPosPerThread;
constexpr uint64_t kEmpty = 0xFFFFFFFFFFFFFFFFull;
constexpr uint32_t kNoSlot = 0xFFFFFFFFu;

struct MineSlot { unsigned long long key; uint32_t count_m1; uint32_t first; };   // memset 0xFF = empty, count 0
static_assert(sizeof(MineSlot) == 16, "slot layout");

struct MineTotals {
    unsigned long long distinct[4];    // tuples per configured order
    unsigned long long found;          // written by the scan: entries that qualify, all orders
    uint32_t error;                    // a probe ran the whole table without finding a place
    uint32_t pad;
    unsigned long long hist[TFE_MINE_HIST_BINS];
};

__device__ __forceinline__ uint64_t mix64(uint64_t x)
{
    x ^= x >> 30; x *= 0xBF58476D1CE4E5B9ull;
    x ^= x >> 27; x *= 0x94D049BB133111EBull;
    x ^= x >> 31;
    return x;
}

// Whole-slot compare-and-swap: {key, count - 1, first} <- put if the slot is still all ones; returns what was there.
__device__ __forceinline__ uint4 cas_empty_slot(MineSlot *slot, unsigned long long key, uint32_t count_m1, uint32_t first)
{
    unsigned long long old_lo, old_hi;
    const unsigned long long put_hi = ((unsigned long long)first << 32) | count_m1;
    asm volatile(
        "{\n\t.reg .b128 o, n, c;\n\t"
        "mov.b128 c, {%2, %3};\n\t"
        "mov.b128 n, {%4, %5};\n\t"
        "atom.global.cas.b128 o, [%6], c, n;\n\t"
        "mov.b128 {%0, %1}, o;\n\t}"
        : "=l"(old_lo), "=l"(old_hi)
        : "l"(kEmpty), "l"(kEmpty), "l"(key), "l"(put_hi), "l"(slot)
        : "memory");
    return make_uint4((uint32_t)old_lo, (uint32_t)(old_lo >> 32), (uint32_t)old_hi, (uint32_t)(old_hi >> 32));
}

// mode 0: ids packed side by side (n * tok_bits <= 63).  mode 1 (n = 4 only): the slots of the bigrams
// ending at t - 2 and at t in the bigram table of this corpus, 31 bits each.
//
// A block takes kCountSpan consecutive end positions.  Equal keys are combined first inside a warp
// (match.any) and then inside the block, in a small shared-memory table {key, count, smallest t}: a frequent
// tuple then costs the global table one update per block instead of one per warp, which is what the hot
// slots of a Zipf-distributed corpus need.  Every distinct key of the block is then looked up / inserted in the
// global table once (the first probes of a thread's entries are issued together); the bigram pass of a wide
// vocabulary also hands every position its slot back through shared memory.
// `cand_slot` (optional, the extraction passes nullptr since its mark pass sweeps the table): the slot for the
// positions that may be a tuple's first occurrence, kNoSlot elsewhere.  The kernel without this bookkeeping
// compiled to 50 registers instead of 48 and ran 7 % slower, so it stays.
constexpr int kCountWin = 2;                               // end positions per thread
constexpr int kCountSpan = kThreads * kCountWin;           // end positions per block
constexpr int kCountEntries = 2 * kCountSpan;              // shared-memory entries: at most half full
constexpr int kEntriesPerThread = kCountEntries / kThreads;

// Six blocks per SM (40 registers): 12.9 ms on the 67 M-id corpus against 13.3 ms at five (48) and 13.3 ms at eight (32, spills).
__global__ void __launch_bounds__(kThreads, 6)
tfe_mine_count_kernel(const int32_t *__restrict__ tokens, uint32_t L, int32_t vocab, int n, int tok_bits, int mode,
                      const uint32_t *__restrict__ pair_slot, MineSlot *table, uint32_t mask,
                      uint32_t *__restrict__ all_slots, uint32_t *__restrict__ cand_slot, MineTotals *totals)
{
    __shared__ unsigned long long s_key[kCountEntries];
    __shared__ uint32_t s_cnt[kCountEntries];              // occurrences in this block; afterwards: 1 if s_min may be the first
    __shared__ uint32_t s_min[kCountEntries];              // smallest end position in this block
    __shared__ uint32_t s_slot[kCountEntries];             // slot in the global table
    for (int e = threadIdx.x; e < kCountEntries; e += kThreads) { s_key[e] = kEmpty; s_cnt[e] = 0; s_min[e] = 0xFFFFFFFFu; }
    __syncthreads();

    const int lane = threadIdx.x & 31;
    const uint32_t base = blockIdx.x * (uint32_t)kCountSpan;
    int entry[kCountWin];
#pragma unroll
    for (int w = 0; w < kCountWin; ++w) {
        const uint32_t t = base + w * kThreads + threadIdx.x;
        bool valid = t < L && t + 1 >= (uint32_t)n;
        unsigned long long key = 0;
        if (valid) {
            if (mode == 0) {
                for (int j = 0; j < n; ++j) {
                    const int32_t x = __ldg(tokens + t - (n - 1) + j);
                    if ((uint32_t)x >= (uint32_t)vocab) valid = false;
                    key = (key << tok_bits) | (uint32_t)x;
                }
            } else {
                const uint32_t a = __ldg(pair_slot + t - 2), b = __ldg(pair_slot + t);
                valid = a != kNoSlot && b != kNoSlot;
                key = ((unsigned long long)a << 31) | b;
            }
        }
        entry[w] = -1;
        const unsigned act = __ballot_sync(0xFFFFFFFFu, valid);
        if (valid) {
            const unsigned grp = __match_any_sync(act, key);
            const int leader = __ffs(grp) - 1;             // lowest lane: the smallest t of the group
            int e = -1;
            if (lane == leader) {
                e = (int)((mix64(key) >> 40) & (kCountEntries - 1));
                for (int probes = 0; probes < kCountEntries; ++probes, e = (e + 1) & (kCountEntries - 1)) {
                    const unsigned long long k = atomicCAS(&s_key[e], kEmpty, key);
                    if (k == kEmpty || k == key) break;
                }
                atomicAdd(&s_cnt[e], (uint32_t)__popc(grp));
                atomicMin(&s_min[e], t);
            }
            entry[w] = __shfl_sync(grp, e, leader);
        }
    }
    __syncthreads();

    // every distinct key of the block, once, against the global table
    unsigned long long keys[kEntriesPerThread];
    uint32_t start[kEntriesPerThread];
    uint4 raw0[kEntriesPerThread];
#pragma unroll
    for (int i = 0; i < kEntriesPerThread; ++i) {
        keys[i] = s_key[threadIdx.x + i * kThreads];
        start[i] = (uint32_t)mix64(keys[i]) & mask;
        if (keys[i] != kEmpty) raw0[i] = __ldcv(reinterpret_cast<const uint4 *>(table + start[i]));
    }
#pragma unroll
    for (int i = 0; i < kEntriesPerThread; ++i) {
        if (keys[i] == kEmpty) continue;
        const int e = threadIdx.x + i * kThreads;
        const unsigned long long key = keys[i];
        const uint32_t t = s_min[e];
        uint32_t slot = kNoSlot, s = start[i];
        uint4 raw = raw0[i];
        bool may_be_first = false;                         // only such positions are looked at by the mark pass
        for (uint32_t probes = 0; probes <= mask; ++probes) {
            // one 16-byte look at the slot: the key and, if it is ours already, the first position so far
            unsigned long long k = ((unsigned long long)raw.y << 32) | raw.x;
            // an empty slot takes the whole entry in one 16-byte compare-and-swap; if another block was
            // faster, the swap returns that block's entry.  (A key whose low word is all ones could be
            // imitated by a half-written slot: the swap then only serves to read the slot atomically.)
            if (k == kEmpty || (k == key && raw.x == 0xFFFFFFFFu)) {
                raw = cas_empty_slot(table + s, key, s_cnt[e] - 1u, t);
                k = ((unsigned long long)raw.y << 32) | raw.x;
                if (k == kEmpty) { slot = s; may_be_first = true; break; }
            }
            if (k == key) {
                slot = s;
                atomicAdd(&table[s].count_m1, s_cnt[e]);
                // `first` only ever decreases: a value already below t needs no update, and t cannot be the first
                if (raw.w > t) { atomicMin(&table[s].first, t); may_be_first = true; }
                break;
            }
            s = (s + 1) & mask;
            raw = __ldcv(reinterpret_cast<const uint4 *>(table + s));
        }
        if (slot == kNoSlot) atomicExch(&totals->error, 1u);
        s_slot[e] = slot;
        s_cnt[e] = may_be_first ? 1u : 0u;
    }
    __syncthreads();

#pragma unroll
    for (int w = 0; w < kCountWin; ++w) {
        const uint32_t t = base + w * kThreads + threadIdx.x;
        if (t >= L) continue;
        const int e = entry[w];
        const uint32_t slot = e >= 0 ? s_slot[e] : kNoSlot;
        if (all_slots) all_slots[t] = slot;
        if (cand_slot) cand_slot[t] = (e >= 0 && s_cnt[e] != 0u && s_min[e] == t) ? slot : kNoSlot;
    }
}

// The table speaks for the tuples: one sequential sweep over its slots.  Every occupied slot is one distinct
// tuple -- counted, added to the histogram of counts and, if its count reaches the threshold, written as
// val[first] = count (val is zero everywhere else).  Sequential reads of the table and a sparse scatter
// replace a random 16-byte read per position.
__global__ void __launch_bounds__(kThreads)
tfe_mine_mark_kernel(const MineSlot *__restrict__ table, uint32_t n_slots, uint32_t min_count, uint32_t *__restrict__ val,
                     MineTotals *totals, int order_index)
{
    __shared__ uint32_t s_hist[TFE_MINE_HIST_BINS];
    __shared__ uint32_t s_distinct;
    for (int i = threadIdx.x; i < TFE_MINE_HIST_BINS; i += kThreads) s_hist[i] = 0;
    if (threadIdx.x == 0) s_distinct = 0;
    __syncthreads();
    const int lane = threadIdx.x & 31;
    uint32_t mine = 0;
    const uint32_t n_round = (n_slots + 31u) & ~31u;
    for (uint32_t s = blockIdx.x * kThreads + threadIdx.x; s < n_round; s += gridDim.x * kThreads) {
        uint4 raw = make_uint4(0xFFFFFFFFu, 0xFFFFFFFFu, 0, 0);
        if (s < n_slots) raw = __ldcs(reinterpret_cast<const uint4 *>(table + s));     // {key lo, key hi, count - 1, first}
        const bool used = (raw.x & raw.y) != 0xFFFFFFFFu;
        const uint32_t count = raw.z + 1u;
        // most tuples of a corpus occur once: those share one histogram update per warp
        const uint32_t ones = __ballot_sync(0xFFFFFFFFu, used && count == 1u);
        if (ones != 0u && lane == __ffs(ones) - 1) atomicAdd(&s_hist[1], __popc(ones));
        if (used) {
            ++mine;
            if (count != 1u) atomicAdd(&s_hist[min(count, (uint32_t)TFE_MINE_HIST_BINS - 1u)], 1u);
            if (count >= min_count) val[raw.w] = count;
        }
    }
    mine = __reduce_add_sync(0xFFFFFFFFu, mine);
    if (lane == 0 && mine) atomicAdd(&s_distinct, mine);
    __syncthreads();
    for (int i = threadIdx.x; i < TFE_MINE_HIST_BINS; i += kThreads)
        if (s_hist[i]) atomicAdd(&totals->hist[i], (unsigned long long)s_hist[i]);
    if (threadIdx.x == 0 && s_distinct) atomicAdd(&totals->distinct[order_index], (unsigned long long)s_distinct);
}

struct MineVals { const uint32_t *val[4]; int n[4]; int n_orders; };

__global__ void __launch_bounds__(kThreads)
tfe_mine_block_sums_kernel(MineVals v, uint32_t L, uint32_t *__restrict__ block_sums)
{
    __shared__ uint32_t s_sum;
    if (threadIdx.x == 0) s_sum = 0;
    __syncthreads();
    uint32_t mine = 0;
    const uint32_t base = blockIdx.x * (uint32_t)kPosPerBlock;
    for (int j = 0; j < kPosPerThread; ++j) {
        const uint32_t t = base + j * kThreads + threadIdx.x;
        if (t < L) {
#pragma unroll
            for (int oi = 0; oi < 4; ++oi)
                if (oi < v.n_orders) mine += __ldg(v.val[oi] + t) != 0u;
        }
    }
    mine = __reduce_add_sync(0xFFFFFFFFu, mine);
    if ((threadIdx.x & 31) == 0 && mine) atomicAdd(&s_sum, mine);
    __syncthreads();
    if (threadIdx.x == 0) block_sums[blockIdx.x] = s_sum;
}

// Exclusive scan of the block totals, one block, running carry; the grand total goes to totals->found.
__global__ void __launch_bounds__(1024)
tfe_mine_scan_kernel(const uint32_t *__restrict__ block_sums, uint32_t n_blocks, unsigned long long *__restrict__ block_offs,
                     unsigned long long *total_out)
{
    __shared__ unsigned long long s_warp[32];
    __shared__ unsigned long long s_carry;
    if (threadIdx.x == 0) s_carry = 0;
    __syncthreads();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (uint32_t base = 0; base < n_blocks; base += 1024) {
        const uint32_t i = base + threadIdx.x;
        const unsigned long long x = i < n_blocks ? block_sums[i] : 0ull;
        unsigned long long incl = x;
        for (int d = 1; d < 32; d <<= 1) {
            const unsigned long long y = __shfl_up_sync(0xFFFFFFFFu, incl, d);
            if (lane >= d) incl += y;
        }
        if (lane == 31) s_warp[warp] = incl;
        __syncthreads();
        if (warp == 0) {
            unsigned long long w = s_warp[lane], wi = w;
            for (int d = 1; d < 32; d <<= 1) {
                const unsigned long long y = __shfl_up_sync(0xFFFFFFFFu, wi, d);
                if (lane >= d) wi += y;
            }
            s_warp[lane] = wi - w;                     // exclusive over warps
        }
        __syncthreads();
        const unsigned long long carry = s_carry;
        if (i < n_blocks) block_offs[i] = carry + s_warp[warp] + incl - x;
        __syncthreads();
        if (threadIdx.x == 1023) s_carry = carry + s_warp[warp] + incl;
        __syncthreads();
    }
    if (threadIdx.x == 0) *total_out = s_carry;
}

// Entry e = (t, oi) in ascending (t, oi) order.  A thread owns kPosPerThread CONSECUTIVE positions here
// (unlike the block-sum kernel, whose per-block totals do not depend on the assignment).
__global__ void __launch_bounds__(kThreads)
tfe_mine_emit_kernel(MineVals v, const int32_t *__restrict__ tokens, uint32_t L,
                     const unsigned long long *__restrict__ block_offs, unsigned long long cap,
                     int32_t *__restrict__ out_tokens, uint8_t *__restrict__ out_len, uint32_t *__restrict__ out_count)
{
    __shared__ uint32_t s_warp[kThreads / 32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t t0 = blockIdx.x * (uint32_t)kPosPerBlock + threadIdx.x * kPosPerThread;
    uint32_t cnt[kPosPerThread][4];
    uint32_t mine = 0;
#pragma unroll
    for (int j = 0; j < kPosPerThread; ++j)
#pragma unroll
        for (int oi = 0; oi < 4; ++oi) {
            cnt[j][oi] = (oi < v.n_orders && t0 + j < L) ? __ldg(v.val[oi] + t0 + j) : 0u;
            mine += cnt[j][oi] != 0u;
        }
    uint32_t incl = mine;
    for (int d = 1; d < 32; d <<= 1) {
        const uint32_t y = __shfl_up_sync(0xFFFFFFFFu, incl, d);
        if (lane >= d) incl += y;
    }
    if (lane == 31) s_warp[warp] = incl;
    __syncthreads();
    uint32_t before = 0;
    for (int w = 0; w < warp; ++w) before += s_warp[w];
    unsigned long long pos = block_offs[blockIdx.x] + before + incl - mine;
    if (mine == 0) return;
#pragma unroll
    for (int j = 0; j < kPosPerThread; ++j)
#pragma unroll
        for (int oi = 0; oi < 4; ++oi) {
            if (cnt[j][oi] == 0u) continue;
            if (pos < cap) {
                const int n = v.n[oi];
                const uint32_t t = t0 + j;
                int4 tup;
                tup.x = n > 0 ? __ldg(tokens + t - (n - 1)) : -1;
                tup.y = n > 1 ? __ldg(tokens + t - (n - 1) + 1) : -1;
                tup.z = n > 2 ? __ldg(tokens + t - (n - 1) + 2) : -1;
                tup.w = n > 3 ? __ldg(tokens + t - (n - 1) + 3) : -1;
                reinterpret_cast<int4 *>(out_tokens)[pos] = tup;
                out_len[pos] = (uint8_t)n;
                out_count[pos] = cnt[j][oi];
            }
            ++pos;
        }
}

// ------------------------------------------------------------------------------------------------
// Initial residency from the counts (paper Sec. 4.3: the GPU tier holds the most frequently accessed entries,
// DRAM the warm ones, SSD the long tail).  The G phrases of largest count are chosen, among equal counts the
// smaller id first; GPU-tier slots are handed out in id order.  key = ~count turns "largest count" into
// "smallest key": three histogram passes (11, 11, 10 bits) find the G-th smallest key and its rank r among the
// phrases that share it; ids are memory order, so the r ties that are in are the first r in memory: per-block
// counts of smaller keys and of ties, their scans, and one pass that numbers the chosen phrases.
constexpr int kResidBins = 2048;

struct ResidState {
    uint32_t hist[kResidBins];
    uint32_t prefix;                // digits of the wanted key chosen so far, in place
    uint32_t k_rem;                 // rank (1-based) of the wanted key among those that share the prefix
    uint32_t ticket;                // blocks done in the current pass
    uint32_t pad;
    unsigned long long total_gt, total_tie, n_host;
};

__global__ void __launch_bounds__(kThreads)
tfe_resid_pass_kernel(const uint32_t *__restrict__ count, uint32_t N, int shift, int bits, uint32_t k_first, int first,
                      ResidState *st)
{
    __shared__ uint32_t s_hist[kResidBins];
    __shared__ uint32_t s_part[kThreads];
    __shared__ uint32_t s_last;
    for (int i = threadIdx.x; i < kResidBins; i += kThreads) s_hist[i] = 0;
    __syncthreads();
    const uint32_t prefix = first ? 0u : st->prefix;
    const int above = shift + bits;
    const uint32_t mask = (1u << bits) - 1u;
    const uint32_t n_round = (N + 31u) & ~31u;
    for (uint32_t i = blockIdx.x * kThreads + threadIdx.x; i < n_round; i += gridDim.x * kThreads) {
        const uint32_t key = i < N ? ~__ldg(count + i) : 0u;
        const bool live = i < N && (above >= 32 || (key >> above) == (prefix >> above));
        const uint32_t digit = (key >> shift) & mask;
        const uint32_t vote = __ballot_sync(0xFFFFFFFFu, live);
        if (live) {
            const uint32_t peers = __match_any_sync(vote, digit);
            if ((threadIdx.x & 31) == __ffs(peers) - 1) atomicAdd(&s_hist[digit], __popc(peers));
        }
    }
    __syncthreads();
    for (int i = threadIdx.x; i < kResidBins; i += kThreads)
        if (s_hist[i]) atomicAdd(&st->hist[i], s_hist[i]);
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) s_last = atomicAdd(&st->ticket, 1u) == gridDim.x - 1;
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    // ---- last block: the digit whose bin holds the wanted rank; the histogram is left zeroed
    constexpr int PER = kResidBins / kThreads;
    uint32_t mine[PER], sum = 0;
#pragma unroll
    for (int j = 0; j < PER; ++j) {
        mine[j] = __ldcg(st->hist + threadIdx.x * PER + j);
        st->hist[threadIdx.x * PER + j] = 0;
        sum += mine[j];
    }
    s_part[threadIdx.x] = sum;
    __syncthreads();
    uint32_t before = 0;
    for (int t = 0; t < (int)threadIdx.x; ++t) before += s_part[t];
    const uint32_t want = first ? k_first : st->k_rem;
    if (want > before && want <= before + sum) {            // exactly one thread
        uint32_t k = want - before;
        int j = 0;
        for (; j < PER - 1 && mine[j] < k; ++j) k -= mine[j];
        st->prefix = prefix | ((uint32_t)(threadIdx.x * PER + j) << shift);
        st->k_rem = k;
    }
    if (threadIdx.x == 0) st->ticket = 0;
}

__global__ void __launch_bounds__(kThreads)
tfe_resid_count_kernel(const uint32_t *__restrict__ count, uint32_t N, const ResidState *st,
                       uint32_t *__restrict__ block_gt, uint32_t *__restrict__ block_tie)
{
    __shared__ uint32_t s_gt, s_tie;
    if (threadIdx.x == 0) { s_gt = 0; s_tie = 0; }
    __syncthreads();
    const uint32_t key_star = st->prefix;
    uint32_t gt = 0, tie = 0;
    const uint32_t base = blockIdx.x * (uint32_t)kPosPerBlock;
    for (int j = 0; j < kPosPerThread; ++j) {
        const uint32_t i = base + j * kThreads + threadIdx.x;
        if (i < N) {
            const uint32_t key = ~__ldg(count + i);
            gt += key < key_star;
            tie += key == key_star;
        }
    }
    gt = __reduce_add_sync(0xFFFFFFFFu, gt);
    tie = __reduce_add_sync(0xFFFFFFFFu, tie);
    if ((threadIdx.x & 31) == 0) { if (gt) atomicAdd(&s_gt, gt); if (tie) atomicAdd(&s_tie, tie); }
    __syncthreads();
    if (threadIdx.x == 0) { block_gt[blockIdx.x] = s_gt; block_tie[blockIdx.x] = s_tie; }
}

// A thread owns kPosPerThread consecutive ids.  chosen = smaller key, or a tie whose rank among all ties (in id
// order) is below r; its slot is the number of chosen phrases before it.
__global__ void __launch_bounds__(kThreads)
tfe_resid_assign_kernel(const uint32_t *__restrict__ count, uint32_t N, ResidState *st, int any_chosen,
                        const unsigned long long *__restrict__ gt_offs, const unsigned long long *__restrict__ tie_offs,
                        uint32_t host_min_count, int32_t *__restrict__ init_slot)
{
    __shared__ uint32_t s_gt[kThreads / 32], s_tie[kThreads / 32], s_host;
    if (threadIdx.x == 0) s_host = 0;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t key_star = st->prefix;
    const unsigned long long r = any_chosen ? st->k_rem : 0ull;
    const uint32_t i0 = blockIdx.x * (uint32_t)kPosPerBlock + threadIdx.x * kPosPerThread;
    uint32_t c[kPosPerThread];
    uint32_t gt = 0, tie = 0;
#pragma unroll
    for (int j = 0; j < kPosPerThread; ++j) {
        c[j] = i0 + j < N ? __ldg(count + i0 + j) : 0u;
        if (i0 + j < N && any_chosen) { gt += ~c[j] < key_star; tie += ~c[j] == key_star; }
    }
    uint32_t gi = gt, ti = tie;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t a = __shfl_up_sync(0xFFFFFFFFu, gi, o), b = __shfl_up_sync(0xFFFFFFFFu, ti, o);
        if (lane >= o) { gi += a; ti += b; }
    }
    if (lane == 31) { s_gt[warp] = gi; s_tie[warp] = ti; }
    __syncthreads();
    unsigned long long gt_before = gt_offs[blockIdx.x] + gi - gt, tie_before = tie_offs[blockIdx.x] + ti - tie;
    for (int w = 0; w < warp; ++w) { gt_before += s_gt[w]; tie_before += s_tie[w]; }
    uint32_t host = 0;
#pragma unroll
    for (int j = 0; j < kPosPerThread; ++j) {
        if (i0 + j >= N) break;
        const uint32_t key = ~c[j];
        const bool is_gt = any_chosen && key < key_star, is_tie = any_chosen && key == key_star;
        int32_t out;
        if (is_gt || (is_tie && tie_before < r)) {
            out = (int32_t)(gt_before + (tie_before < r ? tie_before : r));
        } else {
            out = c[j] >= host_min_count ? -1 : -2;
            host += out == -1;
        }
        init_slot[i0 + j] = out;
        gt_before += is_gt;
        tie_before += is_tie;
    }
    host = __reduce_add_sync(0xFFFFFFFFu, host);
    if (lane == 0 && host) atomicAdd(&s_host, host);
    __syncthreads();
    if (threadIdx.x == 0 && s_host) atomicAdd(&st->n_host, (unsigned long long)s_host);
}

int bits_for(uint32_t max_value)
{
    int b = 1;
    while (b < 32 && (max_value >> b) != 0) ++b;
    return b;
}

uint64_t table_slots_for(int64_t L)
{
    uint64_t want = (uint64_t)std::max<int64_t>(1024, L + L / 2), cap = 1024;
    while (cap < want) cap <<= 1;
    return cap;
}

// Carves the arrays out of one buffer (the caller's, or one allocated here and freed on return).
struct Carver {
    char *base = nullptr, *cur = nullptr, *end = nullptr;
    void *owned = nullptr;
    ~Carver() { if (owned) cudaFree(owned); }
    template <class T> T *take(size_t n)
    {
        const size_t bytes = (std::max<size_t>(n, 1) * sizeof(T) + 255) & ~(size_t)255;
        if (cur + bytes > end) return nullptr;
        T *p = reinterpret_cast<T *>(cur);
        cur += bytes;
        return p;
    }
};

int64_t workspace_bytes_for(int64_t L, int32_t n_orders)
{
    const int64_t n_blocks = (L + kPosPerBlock - 1) / kPosPerBlock;
    const int64_t pad = 256;
    return (int64_t)table_slots_for(L) * (int64_t)sizeof(MineSlot) + pad + (int64_t)(n_orders + 1) * (L * 4 + pad)
           + n_blocks * 12 + 2 * pad + (int64_t)sizeof(MineTotals) + pad + 256;
}

}  // namespace

extern "C" {

int64_t tfe_mine_workspace_bytes(int64_t L, int32_t n_orders)
{
    if (L < 0 || L > TFE_MINE_MAX_TOKENS || n_orders < 1 || n_orders > 4) return -1;
    return workspace_bytes_for(L, n_orders);
}

tfe_status tfe_mine_ngrams(const int32_t *tokens, int64_t L, int32_t vocab, int32_t n_orders, const int32_t *orders,
                           uint32_t min_count, int64_t cap, int32_t *phrase_tokens, uint8_t *phrase_len,
                           uint32_t *phrase_count, int64_t *n_found, int64_t *distinct, int64_t *hist,
                           void *workspace, int64_t workspace_bytes, void *stream_)
{
    if (L < 0 || L > TFE_MINE_MAX_TOKENS || vocab < 1 || n_orders < 1 || n_orders > 4 || !orders || cap < 0 || !n_found)
        return TFE_ERR_INVALID_ARG;
    for (int i = 0; i < n_orders; ++i)
        if (orders[i] < 1 || orders[i] > 4 || (i > 0 && orders[i] <= orders[i - 1])) return TFE_ERR_INVALID_ARG;
    if (L > 0 && !tokens) return TFE_ERR_INVALID_ARG;
    if (cap > 0 && (!phrase_tokens || !phrase_len || !phrase_count)) return TFE_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(phrase_tokens) & 15u) != 0) return TFE_ERR_INVALID_ARG;
    if (workspace_bytes < 0 || (workspace_bytes > 0 && !workspace)) return TFE_ERR_INVALID_ARG;
    if (workspace && workspace_bytes < workspace_bytes_for(L, n_orders)) return TFE_ERR_CAPACITY;
    *n_found = 0;
    if (distinct) for (int i = 0; i < n_orders; ++i) distinct[i] = 0;
    if (hist) for (int i = 0; i < TFE_MINE_HIST_BINS; ++i) hist[i] = 0;
    if (L == 0) return TFE_OK;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
#define MCU(call) do { if ((call) != cudaSuccess) { (void)cudaGetLastError(); return TFE_ERR_CUDA; } } while (0)

    const int tok_bits = bits_for((uint32_t)(vocab - 1));
    const bool composite4 = orders[n_orders - 1] == 4 && 4 * tok_bits > 63;
    const uint64_t slots = table_slots_for(L);
    const uint32_t mask = (uint32_t)(slots - 1);
    const uint32_t n_blocks = (uint32_t)((L + kPosPerBlock - 1) / kPosPerBlock);
    const uint32_t n_count_blocks = (uint32_t)((L + kCountSpan - 1) / kCountSpan);
    int dev_id = 0, sms = 0;
    MCU(cudaGetDevice(&dev_id));
    MCU(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev_id));
    const unsigned mark_grid = (unsigned)std::min<uint64_t>((uint64_t)sms * 8, (slots + kThreads - 1) / kThreads);

    Carver ws;
    if (workspace) {
        ws.base = reinterpret_cast<char *>((reinterpret_cast<uintptr_t>(workspace) + 255) & ~(uintptr_t)255);
        ws.end = static_cast<char *>(workspace) + workspace_bytes;
    } else {
        const int64_t bytes = workspace_bytes_for(L, n_orders);
        MCU(cudaMalloc(&ws.owned, (size_t)bytes));
        ws.base = static_cast<char *>(ws.owned);
        ws.end = ws.base + bytes;
    }
    ws.cur = ws.base;
    MineSlot *table = ws.take<MineSlot>(slots);
    uint32_t *pair_slot = composite4 ? ws.take<uint32_t>((size_t)L) : nullptr;
    uint32_t *block_sums = ws.take<uint32_t>(n_blocks);
    unsigned long long *block_offs = ws.take<unsigned long long>(n_blocks);
    MineTotals *totals = ws.take<MineTotals>(1);
    uint32_t *val[4] = {nullptr, nullptr, nullptr, nullptr};
    bool ok = table && (pair_slot || !composite4) && block_sums && block_offs && totals;
    for (int i = 0; ok && i < n_orders; ++i) ok = (val[i] = ws.take<uint32_t>((size_t)L)) != nullptr;
    if (!ok) return TFE_ERR_INTERNAL;
    MCU(cudaMemsetAsync(totals, 0, sizeof(MineTotals), stream));

    // bigrams first when the 4-grams are keyed by them, even if order 2 itself is not asked for
    std::vector<int> passes;
    if (composite4 && orders[0] != 2 && !(n_orders > 1 && orders[1] == 2)) passes.push_back(-2);
    for (int i = 0; i < n_orders; ++i) passes.push_back(i);
    std::stable_sort(passes.begin(), passes.end(), [&](int a, int b) {
        return (a < 0 ? 2 : orders[a]) < (b < 0 ? 2 : orders[b]);
    });
    for (int pass : passes) {
        const int n = pass < 0 ? 2 : orders[pass];
        const bool keep_pairs = composite4 && n == 2;
        const int mode = (composite4 && n == 4) ? 1 : 0;
        MCU(cudaMemsetAsync(table, 0xFF, slots * sizeof(MineSlot), stream));
        tfe_mine_count_kernel<<<n_count_blocks, kThreads, 0, stream>>>(tokens, (uint32_t)L, vocab, n, tok_bits, mode, pair_slot,
                                                                    table, mask, keep_pairs ? pair_slot : nullptr, nullptr, totals);
        MCU(cudaGetLastError());
        if (pass < 0) continue;
        MCU(cudaMemsetAsync(val[pass], 0, (size_t)L * 4, stream));
        tfe_mine_mark_kernel<<<mark_grid, kThreads, 0, stream>>>(table, (uint32_t)slots, std::max(min_count, 1u), val[pass], totals,
                                                                 pass);
        MCU(cudaGetLastError());
    }
    MineVals mv{};
    mv.n_orders = n_orders;
    for (int i = 0; i < n_orders; ++i) { mv.val[i] = val[i]; mv.n[i] = orders[i]; }
    tfe_mine_block_sums_kernel<<<n_blocks, kThreads, 0, stream>>>(mv, (uint32_t)L, block_sums);
    tfe_mine_scan_kernel<<<1, 1024, 0, stream>>>(block_sums, n_blocks, block_offs, &totals->found);
    tfe_mine_emit_kernel<<<n_blocks, kThreads, 0, stream>>>(mv, tokens, (uint32_t)L, block_offs, (unsigned long long)cap,
                                                          phrase_tokens, phrase_len, phrase_count);
    MCU(cudaGetLastError());
    MineTotals host_totals;
    MCU(cudaMemcpyAsync(&host_totals, totals, sizeof host_totals, cudaMemcpyDeviceToHost, stream));
    MCU(cudaStreamSynchronize(stream));
#undef MCU
    if (host_totals.error) return TFE_ERR_INTERNAL;
    *n_found = (int64_t)host_totals.found;
    if (distinct) for (int i = 0; i < n_orders; ++i) distinct[i] = (int64_t)host_totals.distinct[i];
    if (hist) for (int i = 0; i < TFE_MINE_HIST_BINS; ++i) hist[i] = (int64_t)host_totals.hist[i];
    return TFE_OK;
}

tfe_status tfe_assign_residency(const uint32_t *count, int64_t N, int64_t gpu_slots, uint32_t host_min_count,
                                int32_t *init_slot, int64_t *tiers, void *stream_)
{
    if (N < 0 || N > 0x7FFFFFFFll || gpu_slots < 0 || gpu_slots > 0x7FFFFFFFll) return TFE_ERR_INVALID_ARG;
    if (N > 0 && (!count || !init_slot)) return TFE_ERR_INVALID_ARG;
    const int64_t G = std::min(gpu_slots, N);
    if (tiers) { tiers[0] = G; tiers[1] = 0; tiers[2] = 0; }
    if (N == 0) return TFE_OK;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
#define RCU(call) do { if ((call) != cudaSuccess) { (void)cudaGetLastError(); return TFE_ERR_CUDA; } } while (0)
    const uint32_t n_blocks = (uint32_t)((N + kPosPerBlock - 1) / kPosPerBlock);
    Carver ws;
    const size_t bytes = sizeof(ResidState) + 256 + 2 * ((size_t)n_blocks * 4 + 256) + 2 * ((size_t)n_blocks * 8 + 256) + 256;
    RCU(cudaMalloc(&ws.owned, bytes));
    ws.base = ws.cur = static_cast<char *>(ws.owned);
    ws.end = ws.base + bytes;
    ResidState *st = ws.take<ResidState>(1);
    uint32_t *block_gt = ws.take<uint32_t>(n_blocks), *block_tie = ws.take<uint32_t>(n_blocks);
    unsigned long long *gt_offs = ws.take<unsigned long long>(n_blocks), *tie_offs = ws.take<unsigned long long>(n_blocks);
    if (!st || !block_gt || !block_tie || !gt_offs || !tie_offs) return TFE_ERR_INTERNAL;
    RCU(cudaMemsetAsync(st, 0, sizeof(ResidState), stream));
    int dev = 0, sms = 0;
    RCU(cudaGetDevice(&dev));
    RCU(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    const unsigned grid = (unsigned)std::max<int64_t>(1, std::min<int64_t>((int64_t)sms * 8, (N + kThreads - 1) / kThreads));
    if (G > 0) {
        static const int kShift[3] = {21, 10, 0}, kBits[3] = {11, 11, 10};
        for (int i = 0; i < 3; ++i)
            tfe_resid_pass_kernel<<<grid, kThreads, 0, stream>>>(count, (uint32_t)N, kShift[i], kBits[i], (uint32_t)G, i == 0, st);
        tfe_resid_count_kernel<<<n_blocks, kThreads, 0, stream>>>(count, (uint32_t)N, st, block_gt, block_tie);
        tfe_mine_scan_kernel<<<1, 1024, 0, stream>>>(block_gt, n_blocks, gt_offs, &st->total_gt);
        tfe_mine_scan_kernel<<<1, 1024, 0, stream>>>(block_tie, n_blocks, tie_offs, &st->total_tie);
    } else {
        RCU(cudaMemsetAsync(gt_offs, 0, (size_t)n_blocks * 8, stream));
        RCU(cudaMemsetAsync(tie_offs, 0, (size_t)n_blocks * 8, stream));
    }
    tfe_resid_assign_kernel<<<n_blocks, kThreads, 0, stream>>>(count, (uint32_t)N, st, G > 0 ? 1 : 0, gt_offs, tie_offs,
                                                             host_min_count, init_slot);
    RCU(cudaGetLastError());
    ResidState host_state;
    RCU(cudaMemcpyAsync(&host_state, st, sizeof host_state, cudaMemcpyDeviceToHost, stream));
    RCU(cudaStreamSynchronize(stream));
#undef RCU
    // the selection must account for exactly G phrases: every smaller key plus r of the ties
    if (G > 0 && (host_state.total_gt + host_state.k_rem != (unsigned long long)G || host_state.k_rem > host_state.total_tie))
        return TFE_ERR_INTERNAL;
    if (tiers) { tiers[1] = (int64_t)host_state.n_host; tiers[2] = N - G - (int64_t)host_state.n_host; }
    return TFE_OK;
}

}  // extern "C"
