/*
 * tfe.h -- C ABI of the B200 Engram lookup-and-inject library (libtfe.so).
 *
 * The library implements the per-token side pathway of an Engram-style memory
 * as TF-Engram uses it at inference time: from the token ids ending at each
 * position form the trailing n-gram phrase keys, look each key up in an
 * exact-match (non-colliding) phrase index, decide which matched phrase is
 * retained, see in which storage tier its memory vector lives, fetch the
 * vectors that are in the GPU tier and add them to the hidden state through a
 * gate; phrases whose vectors are not in the GPU tier are reported so the host
 * DRAM / SSD tier and the prefetcher can stage them, and staged vectors are
 * written into the GPU tier by a separate call.
 *
 * Everything below is plain C: opaque context, PODs, raw pointers.  Each
 * pointer is marked HOST or DEVICE.  "stream" is a cudaStream_t passed as
 * void* (NULL = the legacy default stream).  All device work of one context
 * must be issued in stream order (one stream, or streams the caller orders);
 * two calls on the same context that overlap on the GPU race.  A context (and
 * a head) is also not safe for concurrent calls from several host threads:
 * each entry point updates host-side state of its object without locking.
 * Different contexts are independent.
 *
 * No entry point throws, aborts or traps.  Argument errors are found on the
 * host before anything is launched and leave the context unchanged.
 */
#ifndef TFE_H
#define TFE_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct tfe_ctx tfe_ctx;

typedef enum {
    TFE_OK = 0,
    TFE_ERR_INVALID_ARG = 1,
    TFE_ERR_DUPLICATE_PHRASE = 2,   /* two phrases with the same token tuple                    */
    TFE_ERR_KEY_COLLISION = 3,      /* two different tuples of a hashed order share a 64-bit key */
    TFE_ERR_CAPACITY = 4,           /* more phrases than load_factor * index slots, or > 2^32-2 */
    TFE_ERR_SLOT_RANGE = 5,         /* GPU-tier slot outside [0, gpu_slots) or used twice       */
    TFE_ERR_UNKNOWN_PHRASE = 6,
    TFE_ERR_ALREADY_RESIDENT = 7,
    TFE_ERR_MISS_OVERFLOW = 8,      /* caller's miss buffers are smaller than the miss count    */
    TFE_ERR_PROBE_LIMIT = 9,        /* index build could not place a key within max_kicks moves   */
    TFE_ERR_CUDA = 10,              /* a CUDA runtime call failed; see tfe_last_cuda_error()    */
    TFE_ERR_INTERNAL = 11           /* the device reported an inconsistent state or a bounded wait ran out */
} tfe_status;

/* Table geometry, fixed at build time. */
typedef struct {
    int32_t d;                  /* row width in elements; multiple of 8, >= 8                         */
    int32_t vocab;              /* token ids are valid in [0, vocab); anything else is padding        */
    int32_t n_orders;           /* 1..4                                                               */
    int32_t orders[4];          /* n-gram orders, strictly ascending, each in [1,4]                   */
    int64_t n_phrases;          /* N                                                                  */
    int64_t gpu_slots;          /* C, rows of the GPU tier                                            */
    float   load_factor;        /* index slots = ceil(N / load_factor), rounded up to 4-slot buckets  */
    int32_t hidden_dtype;       /* 0 = bf16 hidden states, 1 = fp32 hidden states (rows always bf16)  */
    int32_t max_kicks;          /* cuckoo moves allowed per insertion at build, 0 = default (2000)    */
} tfe_config;

enum { TFE_POLICY_LONGEST = 0, TFE_POLICY_ALL = 1 };
enum { TFE_GATE_CONST = 0, TFE_GATE_COSINE = 1 };
enum { TFE_FLAG_ABSENT = 0, TFE_FLAG_GPU_HIT = 1, TFE_FLAG_HOST_MISS = 2, TFE_FLAG_SSD_MISS = 3 };
#define TFE_NO_PHRASE 0xFFFFFFFFu

/* Per-call injection rule. */
typedef struct {
    int32_t policy;   /* LONGEST: keep the matched phrase of greatest order.  ALL: keep every match
                         and aggregate m = sum_i alpha_i e_i, alpha_i = n_i / sum of matched orders  */
    int32_t gate;     /* CONST: g = lambda.  COSINE: g = lambda * sigmoid(cos(h, m))                 */
    float   lambda;   /* the memory injection scale                                                  */
} tfe_inject_params;

/*
 * tfe_index_build -- build the exact-match phrase index and the per-phrase
 * metadata (paper Sec. 4.2: an index in two levels, from token prefixes to phrase ids and from
 * phrase ids to memory addresses; per phrase its length, the address of its vector, its tier).
 *
 *   cfg            HOST.
 *   phrase_tokens  HOST int32 [N][4]; phrase i is the first phrase_len[i] entries, the rest -1.
 *   phrase_len     HOST uint8 [N]; must be one of cfg->orders.
 *   init_slot      HOST int32 [N]; >= 0: GPU-tier slot holding the vector; -1: host DRAM; -2: SSD.
 *   gpu_rows       DEVICE bf16 [C][d] row-major, 16-byte aligned, CALLER-OWNED, already holding
 *                  the vectors of the resident phrases.  The library keeps the pointer and writes
 *                  to it only in tfe_cache_install.
 *   stream         work is issued here; the call synchronises it before returning.
 *   out            receives the context (phrase id = index into the arrays above).
 *
 * Errors (nothing is kept): INVALID_ARG (geometry, length not an order, token outside [0,vocab)),
 * DUPLICATE_PHRASE, KEY_COLLISION, CAPACITY, SLOT_RANGE, PROBE_LIMIT, CUDA.
 */
tfe_status tfe_index_build(const tfe_config *cfg, const int32_t *phrase_tokens,
                           const uint8_t *phrase_len, const int32_t *init_slot, void *gpu_rows,
                           void *stream, tfe_ctx **out);

/*
 * tfe_index_build_device -- the same construction with the phrase table already on the DEVICE
 * (phrase_tokens int32 [N][4] 16-byte aligned, phrase_len uint8 [N], init_slot int32 [N]) and
 * every step on the GPU: key formation and input checks, two-choice cuckoo placement with
 * 128-bit compare-and-swap / exchange on whole index slots, and a final pass in which every
 * phrase looks itself up (which is also how equal tuples and colliding hashes are found).  The
 * paper's index construction is its dominant offline cost (Sec. 5.3); this is that step for
 * tables that are produced or kept on the GPU.  Results of later calls do not depend on which
 * of the two builds made the context (only the mapping is defined, not the slot a key sits in).
 * Two kernel launches, one synchronisation of `stream`; the host-side copy of the residency
 * state that tfe_cache_install checks its arguments against is fetched on its first call.
 * Errors as tfe_index_build; when several problems are present
 * the one reported may differ.
 */
tfe_status tfe_index_build_device(const tfe_config *cfg, const int32_t *phrase_tokens,
                                  const uint8_t *phrase_len, const int32_t *init_slot,
                                  void *gpu_rows, void *stream, tfe_ctx **out);

/*
 * tfe_cache_install -- write n fetched vectors into GPU-tier slots and make
 * their phrases GPU-resident (paper Sec. 4.3: an entry read from DRAM / SSD is
 * inserted into a faster tier when it arrives; Sec. 4.4: prefetched entries
 * are moved into the GPU cache before they are needed).
 *
 *   phrase_ids  HOST uint32 [n]; valid, pairwise distinct, currently NOT GPU-resident.
 *   src_rows    bf16 [n][d]; HOST (pinned memory makes the copy asynchronous; it must stay valid
 *               until the stream has passed this call) or DEVICE.
 *   dst_slots   HOST int32 [n]; pairwise distinct, in [0, C).  A slot that holds another phrase
 *               is overwritten and that phrase falls back to the host-DRAM tier.
 *   Asynchronous on `stream`; a lookup issued later on the same stream sees the new state.
 *   phrase_ids / dst_slots may be reused as soon as the call returns.
 *
 * Errors (state unchanged): INVALID_ARG, UNKNOWN_PHRASE, ALREADY_RESIDENT, SLOT_RANGE, CUDA.
 */
tfe_status tfe_cache_install(tfe_ctx *ctx, int32_t n, const uint32_t *phrase_ids,
                             const void *src_rows, const int32_t *dst_slots, void *stream);

/*
 * tfe_cache_install_device -- the same insertion with the whole batch on the DEVICE and no check
 * by the host: what a prefetch loop that stays on the GPU produces (candidate phrases from
 * tfe_prefetch_candidates, destination slots from tfe_cache_select_victims_device, rows staged in
 * device memory).  Entries that cannot be applied are skipped instead of refusing the batch.
 * Judged against the state before the call, entry k is a candidate if phrase_ids[k] is a phrase,
 * that phrase is not GPU-resident, dst_slots[k] is a slot and no earlier entry names the same
 * phrase; it is applied if in addition no earlier candidate names the same slot.  Applied
 * entries take effect as in tfe_cache_install.
 *
 *   n              0..4096
 *   phrase_ids     DEVICE uint32 [n];  src_rows DEVICE [n][d] bf16, 16-byte aligned;
 *   dst_slots      DEVICE int32 [n]
 *   applied        DEVICE uint8 [n], receives 1 / 0 per entry, or NULL
 *   applied_count  DEVICE uint32, receives the number applied, or NULL
 * Asynchronous on `stream`, two kernel launches, never synchronises.  The first call on a context
 * allocates 4 bytes per phrase and per slot (with a device synchronisation: make it outside a stream
 * capture); every later call keeps no state on the host and may be captured into a CUDA graph and
 * replayed with new contents in the same buffers.  Once this function has been used, the host-side
 * residency copy that tfe_cache_install checks against is re-read from the device (one
 * synchronisation) on every call of that function.
 * Errors: INVALID_ARG, CUDA.
 */
tfe_status tfe_cache_install_device(tfe_ctx *ctx, int32_t n, const uint32_t *phrase_ids,
                                    const void *src_rows, const int32_t *dst_slots, uint8_t *applied,
                                    uint32_t *applied_count, void *stream);

/*
 * tfe_lookup_inject -- the hot path, one kernel launch (paper Sec. 2.2: key
 * from token n-grams, lookup m_t = M(q_t), aggregation m_t = sum alpha_i v_i,
 * injection h'_t = h_t + g_t * m_t; Sec. 4.2: longest-match selection;
 * Sec. 4.3: tier walk).
 *
 *   tokens      DEVICE int32 [B][T] row-major.
 *   q_start     queries are the positions t in [q_start, T) of every sequence,
 *               numbered q = b*(T-q_start) + (t-q_start); Q = B*(T-q_start).  An n-gram ends at
 *               its query position and never reaches before t = 0 of its sequence.
 *   h           DEVICE [Q][d] hidden states (bf16 or fp32 per cfg.hidden_dtype), 16-byte aligned.
 *   out         DEVICE [Q][d], same dtype; may be the same pointer as h (then only injected
 *               positions are touched); must not partially overlap h.
 *   params      HOST.
 *   sel_phrase  DEVICE uint32 [Q] (LONGEST) or [Q][n_orders] (ALL, column = index into orders);
 *   sel_slot    DEVICE int32, same shape: slot (hit), -1 host, -2 SSD, -3 absent;
 *   flags       DEVICE uint8, same shape: TFE_FLAG_*.   Any of the three may be NULL.
 *
 * Positions whose retained phrase is GPU-resident get out = round(h + g*m) (fp32 arithmetic,
 * round-to-nearest-even into the hidden dtype); every other position gets out = h bit for bit.
 * A retained phrase that is not GPU-resident is NOT replaced by a shorter resident one; it goes to
 * the miss list.  Asynchronous; launches exactly one kernel and never synchronises.
 * Errors: INVALID_ARG, CUDA (a first call with a larger Q than any before grows context buffers).
 */
tfe_status tfe_lookup_inject(tfe_ctx *ctx, const int32_t *tokens, int32_t B, int32_t T,
                             int32_t q_start, const void *h, void *out,
                             const tfe_inject_params *params, uint32_t *sel_phrase,
                             int32_t *sel_slot, uint8_t *flags, void *stream);

/*
 * tfe_lookup_inject_host -- the same call for HOST buffers (tokens, h, out and the optional
 * result arrays all in host memory; pinned memory lets the copies run asynchronously and
 * overlap): copies the inputs to context-owned device buffers, runs the kernel, copies the
 * results back, without synchronising the host.  Everything is ordered after the work already
 * queued on `stream`, and `stream` continues only when the last result byte is in host memory,
 * so the caller sees the call as one operation on `stream`.  The buffers must stay valid until
 * the stream has passed the call.
 *
 * LONGEST / CONST calls with at least 16 MiB of hidden state are issued in pieces (query ranges;
 * up to 32, small at both ends, up to 8 MiB in the middle) through two context-owned copy
 * streams, so that one piece's kernel runs while the next piece comes in and the previous one
 * goes back; the last piece's launch builds the miss list of the whole call.  Results are the
 * same as for the single launch.  Other variants copy, launch once and copy back on `stream`.
 * The first piecewise call on a context creates the two streams and their events.
 */
tfe_status tfe_lookup_inject_host(tfe_ctx *ctx, const int32_t *tokens, int32_t B, int32_t T,
                                  int32_t q_start, const void *h, void *out,
                                  const tfe_inject_params *params, uint32_t *sel_phrase,
                                  int32_t *sel_slot, uint8_t *flags, void *stream);

/*
 * tfe_miss_list -- the compacted, order-stable list of retained phrases that were not
 * GPU-resident in the most recent lookup of this context (paper Sec. 4.3: such entries are staged
 * from DRAM or read asynchronously from SSD; Sec. 4.4: the prefetcher consumes the same records).
 * Entries are in ascending (q, order); duplicates are kept; tier is TFE_FLAG_HOST_MISS / SSD_MISS.
 *
 *   q_idx, phrase_id, tier   HOST buffers of `cap` entries (may be NULL if cap == 0).
 *   count                    HOST, always receives the full miss count.
 *   Synchronises `stream`.  Errors: MISS_OVERFLOW (count > cap; the first cap entries are
 *   returned), INTERNAL, CUDA.
 */
tfe_status tfe_miss_list(tfe_ctx *ctx, uint32_t *q_idx, uint32_t *phrase_id, uint8_t *tier,
                         int64_t cap, int64_t *count, void *stream);

/*
 * tfe_lookup_inject_noalloc -- tfe_lookup_inject for callers that must not allocate.  (The paper
 * has no counterpart for this entry point; it exists for the sake of the embedding runtime.)
 *
 * tfe_lookup_inject lets the context cudaMalloc its per-call scratch on first use and again when
 * a larger call arrives.  A runtime that has given all free device memory to its own pool, or a
 * latency-critical loop that cannot tolerate the device-wide synchronisation an allocation or a
 * free brings, calls this instead: it allocates and frees nothing, on the host or on the device.
 * Its scratch is a fixed area inside the loaded library image (2 MiB: one 8-byte result record per
 * entry; present on every GPU that loads the library until the process ends), which bounds the call:
 *
 *     Q * (policy == ALL ? n_orders : 1)  <=  262,144      otherwise TFE_ERR_CAPACITY.
 *
 *   tokens ... flags   as for tfe_lookup_inject (DEVICE; sel_phrase / sel_slot / flags may be NULL).
 *   miss_q, miss_phrase, miss_tier
 *                      DEVICE, CALLER-OWNED, each with room for Q * (ALL ? n_orders : 1) entries;
 *                      receive the ordered miss list (the context's own list and tfe_miss_list are
 *                      not involved).  Required.
 *   miss_count         DEVICE uint32, receives the number of entries written.  Required.
 *
 * The context's device must be the current device.  The first call on a device looks up the
 * address of the scratch area (cudaGetSymbolAddress); make that first call outside any stream
 * capture.  All calls on one device share the area, whatever their context, and it keeps what the
 * last call left: a call puts the launch state back to zero on its stream (a call refused for its
 * arguments touches nothing), and records carry the number of the call that wrote them, so a record
 * left by an earlier call is never taken for one of this call.  Two calls that overlap on the GPU
 * (different streams, no dependency) race.  Results are those of tfe_lookup_inject.
 * Errors: INVALID_ARG, CAPACITY, CUDA.
 */
tfe_status tfe_lookup_inject_noalloc(tfe_ctx *ctx, const int32_t *tokens, int32_t B, int32_t T,
                                     int32_t q_start, const void *h, void *out,
                                     const tfe_inject_params *params, uint32_t *sel_phrase,
                                     int32_t *sel_slot, uint8_t *flags, uint32_t *miss_q,
                                     uint32_t *miss_phrase, uint8_t *miss_tier, uint32_t *miss_count,
                                     void *stream);

/* The same list as DEVICE pointers owned by the context, valid until the next lookup; no sync. */
tfe_status tfe_miss_list_device(tfe_ctx *ctx, const uint32_t **q_idx, const uint32_t **phrase_id,
                                const uint8_t **tier, const uint32_t **count);

/*
 * GPU-tier retention ranking (paper Sec. 4.3 names the signals an implementation may rank entries by --
 * access frequency and recency among them -- and gives no formula; the ranking below is this
 * library's reading).
 *
 * tfe_cache_policy_enable -- starts the bookkeeping: from now on every lookup of this context
 * (tfe_lookup_inject, tfe_lookup_inject_host; not tfe_lookup_inject_noalloc) adds 1 to `freq` and
 * stores the call's epoch in `last` for every GPU-tier slot it injects from, and every
 * tfe_cache_install sets {freq, last} = {1, epoch} for the slots it fills.  The epoch is a device
 * counter of completed lookups (a replayed launch advances it like a fresh one).  Calling it
 * again clears the counters and the epoch.  Allocates 8 bytes per GPU-tier slot and 8.2 MiB of work
 * space for the selection on the first call; waits for the device then.  Launches recorded earlier (a captured CUDA graph) keep the arguments they were
 * recorded with and do no bookkeeping; record them again after enabling.
 * Errors: INVALID_ARG, CUDA.
 */
tfe_status tfe_cache_policy_enable(tfe_ctx *ctx, void *stream);

/*
 * tfe_cache_select_victims -- the n slots least worth keeping at the current epoch `now`:
 *     age     = now - last                                  (unsigned 32-bit)
 *     decayed = freq >> min(31, age / half_life)            (half_life <= 0: no decay)
 *     key     = min(decayed, 65535) << 16 | (65535 - min(age, 65535));  key = 0 for a free slot
 * in ascending (key, slot): free slots first, then by decayed frequency, ties by least recent
 * use, then by slot.  half_life -> large gives least-frequently-used order, equal frequencies
 * give least-recently-used order.
 *
 *   n        0..4096;  half_life at most 2^26 - 1;  slots HOST int32 [n], or NULL;  keys HOST uint32 [n] or NULL;
 *   count    HOST: entries written = min(n, gpu_slots).
 * One cooperative kernel launch on `stream` (one block per SM; its blocks wait for one another at
 * two or more step boundaries, every wait bounded).  The
 * per-slot bookkeeping is read once; a threshold taken from a sample of the slots keeps the work
 * after that pass to a candidate list, and the result does not depend on the sample: a threshold
 * that turns out too low or too high only makes the call walk the table again.  With host `slots`
 * the results are copied there and the stream is synchronised (they feed tfe_cache_install, which
 * takes host arrays); with slots = NULL nothing is copied and nothing synchronises.
 * tfe_cache_select_victims_device returns the DEVICE copies of the most recent selection (owned
 * by the context, valid until the next one; they feed tfe_cache_install_device).
 * One selection at a time per context (the work space is the context's).
 * Errors: INVALID_ARG (also: policy not enabled, half_life too large), CUDA, INTERNAL (a wait inside the
 * kernel ran out or its counts contradicted one another; the outputs are not valid.  Reported by the
 * form with host `slots`, which also clears the condition; until then later selections do nothing).
 */
tfe_status tfe_cache_select_victims(tfe_ctx *ctx, int32_t n, int32_t half_life, int32_t *slots,
                                    uint32_t *keys, int32_t *count, void *stream);
tfe_status tfe_cache_select_victims_device(tfe_ctx *ctx, const int32_t **slots, const uint32_t **keys);

/*
 * tfe_cache_select_tuning -- sizes of the selection's internal steps, for tests and tuning; the
 * result of tfe_cache_select_victims does not depend on them.  list_cap: entries of the candidate
 * list (1..1048576), final_cap: numbers the last step ranks (..8192; at least n + 1 is used; a table
 * with more slots than either is sampled for a threshold), n_samples: slots sampled
 * (..2048).  0 or less: the default.  Takes effect with the next selection.
 * Errors: INVALID_ARG.
 */
tfe_status tfe_cache_select_tuning(tfe_ctx *ctx, int32_t list_cap, int32_t final_cap, int32_t n_samples);

/*
 * tfe_cache_stats -- copies the bookkeeping to the host: freq_last HOST uint32 [gpu_slots][2]
 * ({freq, last} per slot) and/or the epoch (either may be NULL).  Synchronises `stream`.
 */
tfe_status tfe_cache_stats(tfe_ctx *ctx, uint32_t *freq_last, uint32_t *epoch, void *stream);

/* Scoring of prefetch candidates. */
typedef struct {
    float   benefit_host;   /* c_i of an entry that sits in host DRAM (>= 0)                           */
    float   benefit_ssd;    /* c_i of an entry that sits only on SSD (>= 0); GPU-resident entries: 0   */
    int32_t budget;         /* at most this many candidates are returned, 0..4096                      */
} tfe_prefetch_params;

/*
 * tfe_prefetch_candidates -- candidate phrase expansion and priority for early-exit guided
 * prefetching (paper Sec. 4.4: each predicted token is put behind the sequence's recent history, the
 * n-grams that result are looked up in the token-to-phrase index and give the candidate set Q_t;
 * a candidate's priority is s_i = p_i * r_i * c_i, and the budget goes to the highest priorities,
 * the rest is dropped).  The top-K tokens and their probabilities are inputs: they come from the
 * early-exit head, tfe_head_topk below, or from anywhere else.
 *
 *   history      DEVICE int32 [B][H]: the last H tokens of every sequence (H >= n_max - 1 to let
 *                every order contribute; an order n with n - 1 > H contributes nothing).
 *   cand_tokens  DEVICE int32 [B][K]: predicted next tokens;  cand_prob DEVICE float [B][K]: p.
 *   usefulness   DEVICE float [N]: r of every phrase, or NULL for r = 1.
 *   params       HOST.
 * For every sequence b, token k and configured order n the n-gram (history[b][H-n+1..H-1],
 * cand_tokens[b][k]) is looked up; a phrase found outside the GPU tier is a candidate with
 * s = (p * r) * c in fp32, dropped if s <= 0.  Outputs (DEVICE, `budget` entries each): phrase id,
 * tier (TFE_FLAG_HOST_MISS / TFE_FLAG_SSD_MISS), s, and source b*K + k of the `budget` best, in
 * descending s, equal s in ascending (b, k, order); duplicates of one phrase are kept.
 * out_count DEVICE uint32 [2]: entries written, candidates found before the cut.  The phrase ids
 * beyond the entries written are set to TFE_NO_PHRASE (the other arrays are left as they were), so
 * the whole array can be handed to tfe_cache_install_device, which skips ids that are no phrase.
 * Asynchronous on `stream`, two kernel launches; a first call with more entries than any before
 * grows context buffers.  Errors: INVALID_ARG, CUDA.
 */
tfe_status tfe_prefetch_candidates(tfe_ctx *ctx, const int32_t *history, int32_t B, int32_t H,
                                   const int32_t *cand_tokens, const float *cand_prob, int32_t K,
                                   const float *usefulness, const tfe_prefetch_params *params,
                                   uint32_t *out_phrase, uint8_t *out_tier, float *out_score,
                                   uint32_t *out_src, uint32_t *out_count, void *stream);

/* Frees everything the context owns (not gpu_rows).  NULL is allowed. */
void tfe_destroy(tfe_ctx *ctx);

const char *tfe_status_string(tfe_status s);

/* Text of the last CUDA error seen by this thread's calls ("" if none). */
const char *tfe_last_cuda_error(void);

/*
 * Introspection used by tests and the benchmark (HOST only, no device work).
 *   tfe_index_geometry  buckets (of 4 slots of 16 bytes), bytes of the device index, bytes of per-phrase metadata.
 *   tfe_phrase_key64    the 64-bit index key of a token tuple (0 if n or a token is invalid) and
 *                       whether that order is packed injectively (exact) or hashed + verified.
 *   tfe_home_bucket     the first bucket probed for a key.
 *   tfe_launch_geometry grid size, block size and queries per warp round of the last lookup.
 */
tfe_status tfe_index_geometry(const tfe_ctx *ctx, int64_t *n_buckets, int64_t *index_bytes,
                              int64_t *metadata_bytes);
uint64_t tfe_phrase_key64(int32_t vocab, const int32_t *tokens, int32_t n, int32_t *is_exact);
uint64_t tfe_home_bucket(uint64_t key, uint64_t n_buckets);
tfe_status tfe_launch_geometry(const tfe_ctx *ctx, int32_t *grid, int32_t *block, int32_t *batch_queries);

/*
 * Tuning knob (HOST only; results never depend on it).  A lookup warp takes batches of 1..8
 * consecutive queries: it probes the whole batch at once (one lane per query and order), then
 * streams the batch's rows.  0 = the library picks per call (small calls 1, the lowest latency;
 * large calls 4).
 */
tfe_status tfe_set_tuning(tfe_ctx *ctx, int32_t batch_queries);

/*
 * Early-exit prefetch head (paper Sec. 4.4): p_early(x_{t+1} | x_<=t) = softmax(W_pref h_t^{L-r})
 * and T_early = TopK(p_early) -- the K most likely next tokens of every sequence with their
 * probabilities, which are the inputs of tfe_prefetch_candidates.  The only dense contraction of
 * the method; it runs on the tensor cores.  A head is independent of any phrase index.
 *
 * tfe_head_create -- w_pref DEVICE bf16 [V][d] row-major, 16-byte aligned, CALLER-OWNED; it is
 * copied into the head in the order the GEMM reads it (pieces of 128 rows x 64 columns, 16
 * contiguous KB each) and may be released when the call returns (the call waits for the device);
 * d a multiple of 64; max_batch 1..256.  Allocates that copy (V * d * 2 bytes, rounded up to
 * whole 128-row tiles per CTA: 349 MB for V = 151,936, d = 1,024), the logits buffer
 * (max_batch * V * 4 bytes) and small work areas on the current device.
 * Errors: INVALID_ARG, CUDA.
 */
typedef struct tfe_head tfe_head;
tfe_status tfe_head_create(const void *w_pref, int32_t V, int32_t d, int32_t max_batch, tfe_head **out);
void       tfe_head_destroy(tfe_head *head);

/*
 * tfe_head_topk -- hidden DEVICE bf16 [B][d] (16-byte aligned), 0 <= B <= max_batch, 1 <= K <= 128,
 * K <= V.  Outputs DEVICE: cand_tokens int32 [B][K], cand_prob float [B][K], per sequence in
 * descending probability, equal logits in ascending token id.  Logits are bf16 products
 * accumulated in fp32 (tensor cores); selection and softmax in fp32.  Asynchronous on `stream`,
 * two kernel launches, never synchronises.  Errors: INVALID_ARG, CUDA, INTERNAL.
 */
tfe_status tfe_head_topk(tfe_head *head, const void *hidden, int32_t B, int32_t K, int32_t *cand_tokens,
                         float *cand_prob, void *stream);

/* DEVICE views of the most recent call: logits fp32 [B][ld] and log-sum-exp fp32 [B]; owned by the head. */
tfe_status tfe_head_buffers(tfe_head *head, const float **logits, int64_t *ld, const float **lse);

/*
 * tfe_head_status -- synchronises `stream` and reads the device status word: 0, or a bit set by a
 * wait inside the kernel that ran out (1 loader, 2 MMA issuer, 4 epilogue); then INTERNAL.
 */
tfe_status tfe_head_status(tfe_head *head, uint32_t *device_flags, void *stream);

/* Launch geometry: CTAs, vocabulary rows per CTA, rows of each CTA's short last tile. */
tfe_status tfe_head_geometry(const tfe_head *head, int32_t *grid, int32_t *rows_per_cta, int32_t *tail_rows);

/*
 * N-gram extraction with a frequency threshold (paper Sec. 4.2, construction pipeline: candidate
 * phrases such as bigrams and trigrams are selected by a frequency threshold; Sec. 5.3: this
 * tokenizer-level n-gram extraction dominates the offline cost of building a table).  Independent of
 * any context; its output is the phrase table that tfe_index_build_device takes.
 *
 *   tokens         DEVICE int32 [L], the tokenised corpus; an id outside [0, vocab) separates documents:
 *                  no window contains one.  0 <= L <= TFE_MINE_MAX_TOKENS.
 *   orders         HOST int32 [n_orders], strictly ascending, each in 1..4.
 *   window         for an order n and an end position t >= n - 1 whose n ids x_{t-n+1} .. x_t are all
 *                  valid, that tuple occurs once at t.  count(tuple) = number of occurrences,
 *                  first(tuple) = its smallest end position.
 *   result         the tuples with count >= min_count (0 means 1) in ascending (first, n) order:
 *                  phrase_tokens DEVICE int32 [cap][4] (16-byte aligned; unused trailing ids -1),
 *                  phrase_len DEVICE uint8 [cap], phrase_count DEVICE uint32 [cap]; may be NULL if cap = 0.
 *   n_found        HOST: how many tuples qualify; min(n_found, cap) entries were written (the first ones
 *                  in that order) -- n_found > cap is not an error, the caller raises min_count or cap.
 *   distinct       HOST int64 [n_orders] or NULL: different tuples per order.
 *   hist           HOST int64 [TFE_MINE_HIST_BINS] or NULL: hist[c] = different tuples, all orders together,
 *                  that occur exactly c times; the last bin collects every c >= TFE_MINE_HIST_BINS - 1.
 *                  sum_{c >= m} hist[c] is n_found for min_count = m, so one call tells which threshold
 *                  yields a table of a wanted size.
 *
 *   workspace      DEVICE scratch of workspace_bytes >= tfe_mine_workspace_bytes(L, n_orders) (about 24..48
 *                  bytes per token for the counting table plus 4 bytes per token and order (+ 1); smaller:
 *                  TFE_ERR_CAPACITY), contents undefined before and after; or NULL with workspace_bytes = 0:
 *                  the call allocates and frees it (several milliseconds per call at 10^8 tokens).
 *
 * Launches on `stream` and synchronises it.  Exact for every vocabulary: orders whose ids do not fit one
 * 64-bit key side by side are keyed through the exact names of their halves.  Errors:
 * TFE_ERR_INVALID_ARG, TFE_ERR_CAPACITY, TFE_ERR_CUDA (the workspace could not be allocated),
 * TFE_ERR_INTERNAL (a bounded probe ran out).
 */
#define TFE_MINE_HIST_BINS 1024
#define TFE_MINE_MAX_TOKENS (1ll << 30)
tfe_status tfe_mine_ngrams(const int32_t *tokens, int64_t L, int32_t vocab, int32_t n_orders, const int32_t *orders,
                           uint32_t min_count, int64_t cap, int32_t *phrase_tokens, uint8_t *phrase_len,
                           uint32_t *phrase_count, int64_t *n_found, int64_t *distinct, int64_t *hist,
                           void *workspace, int64_t workspace_bytes, void *stream);
int64_t tfe_mine_workspace_bytes(int64_t L, int32_t n_orders);   /* -1 for invalid arguments */

/*
 * Initial residency from corpus counts (paper Sec. 4.3: the GPU tier is reserved for the most frequently
 * accessed entries, DRAM holds warm entries, SSD absorbs the long tail).  Turns the counts that
 * tfe_mine_ngrams returns into the init_slot array that tfe_index_build_device takes.
 *
 *   count           DEVICE uint32 [N];  init_slot DEVICE int32 [N] (output);  0 <= N, gpu_slots < 2^31
 *   rule            the G = min(gpu_slots, N) phrases of largest count start in the GPU tier, among equal
 *                   counts the smaller id first; GPU-tier slots are handed out in id order (the chosen
 *                   phrase with the k-th smallest id gets slot k).  Of the others, count >= host_min_count
 *                   means host DRAM (-1), a smaller count SSD (-2).
 *   tiers           HOST int64 [3] or NULL: phrases per tier (GPU, host, SSD).
 *
 * Allocates a few bytes per 1,024 phrases, launches on `stream`, synchronises it.
 * Errors: TFE_ERR_INVALID_ARG, TFE_ERR_CUDA, TFE_ERR_INTERNAL (the selection's totals do not add up).
 */
tfe_status tfe_assign_residency(const uint32_t *count, int64_t N, int64_t gpu_slots, uint32_t host_min_count,
                                int32_t *init_slot, int64_t *tiers, void *stream);

/*
 * Streaming copy (the paper has no counterpart: a yardstick for the measurements, not a step of the method).
 * Copies `bytes` bytes from `src` to `dst` (DEVICE, 16-byte aligned, bytes a multiple of 16, ranges must not
 * overlap) with the load / store instructions the lookup kernels stream hidden states with, one asynchronous
 * launch on `stream`, graph-capturable.  The benchmark times it on a transfer of the lookup call's own footprint:
 * what a plain copy of that many bytes reaches on the device is the ceiling the lookup's rate is read against.
 * Errors: TFE_ERR_INVALID_ARG, TFE_ERR_CUDA.
 */
tfe_status tfe_stream_copy(void *dst, const void *src, int64_t bytes, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* TFE_H */
