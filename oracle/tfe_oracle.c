/*
 * tfe_oracle.c -- plain CPU oracle for the Engram lookup-and-inject step.
 *
 * TEST INFRASTRUCTURE, NOT PRODUCT CODE.  Only the tests, the smoke check and
 * the benchmark's CPU-baseline / reference legs may build, load or call this
 * file.  It shares no code, header, table or constant with the CUDA library
 * and includes nothing from it.  It is written for the eye, not for speed:
 * every function is the definition it cites, written out as loops over plain
 * arrays, floating point in double.  The only parallelism is one optional
 * OpenMP "parallel for" over independent query positions.
 *
 * What it computes (paper sections in brackets):
 *   - trailing n-gram phrase keys of a token stream          [Sec. 2.2, Sec. 4.2]
 *   - exact phrase match against a table of token tuples     [Sec. 4.2, two-level index]
 *   - longest-match selection / all-match retention          [Sec. 4.2, selection policy]
 *   - tier walk GPU / host DRAM / SSD                         [Sec. 4.3, memory hierarchy]
 *   - aggregation  m_t = sum_i alpha_i e_i                    [Sec. 2.2 aggregation eq.; Sec. 4.2 e_phi eq.]
 *   - gated residual injection  h'_t = h_t + g_t * m_t        [Sec. 2.2 injection eq.]
 *   - list of matched-but-not-GPU-resident phrases            [Sec. 4.3, staged / asynchronous reads]
 *   - insertion of fetched entries into the GPU tier          [Sec. 4.3, promotion of a fetched entry into a faster tier]
 *   - prefetch candidates from predicted tokens + priority     [Sec. 4.4, candidate set Q_t, score s = p r c]
 *   - retention ranking of GPU-tier slots (frequency, recency) [Sec. 4.3, cache policy signals]
 *   - early-exit prefetch head: softmax(W_pref h), top-K        [Sec. 4.4, p_early and T_early equations]
 *   - n-gram extraction with a frequency threshold              [Sec. 4.2, construction pipeline; Sec. 5.3]
 *   - initial residency from corpus counts                      [Sec. 4.3, tiers by access frequency]
 *
 * Parity pins: every function here is pinned by tests that do not call it to
 * produce their expected values (hand-made cases, closed forms, a library
 * conversion routine, brute force) EXCEPT the COSINE gate away from its
 * special cases (m = h, m = -h, m orthogonal to h, m = 0): the paper leaves the
 * form of the gate open (Sec. 2.2), so the formula
 * g = lambda * sigmoid(cos(h, m)) is this build's own reading --
 * COSINE gate: parity unpinned.
 * The same holds for the retention ranking: the paper lists its signals and no formula, so the
 * key (decayed frequency, then recency) is this build's reading, pinned only where it reduces to
 * textbook least-recently-used / least-frequently-used order -- retention ranking: parity unpinned.
 *
 * Conventions shared by all functions
 *   tokens        int32 [B][T] row-major.  Ids outside [0, vocab) are padding:
 *                 an n-gram containing one matches nothing.
 *   query index   q = b * (T - q_start) + (t - q_start), t in [q_start, T).
 *   phrase table  phrase_tokens int32 [N][4] (unused trailing entries = -1),
 *                 phrase_len uint8 [N]; tuples are pairwise distinct.
 *   residency     slot_state int32 [N]: >= 0 GPU-tier slot, -1 host DRAM, -2 SSD.
 *   rows          bf16 bit patterns (uint16) [C][d] row-major, the GPU tier.
 *   flags         0 absent, 1 GPU hit (injected), 2 host miss, 3 SSD miss.
 *   sel_slot      slot for a GPU hit, -1 / -2 for a miss, -3 for absent.
 *   sel_phrase    phrase id, 0xFFFFFFFF for absent.
 */
#define _GNU_SOURCE     /* qsort_r */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORC_ABSENT_PHRASE 0xFFFFFFFFu
#define ORC_MAX_ORDERS 4

enum { ORC_POLICY_LONGEST = 0, ORC_POLICY_ALL = 1 };
enum { ORC_GATE_CONST = 0, ORC_GATE_COSINE = 1 };
enum { ORC_HIDDEN_BF16 = 0, ORC_HIDDEN_F32 = 1 };

int orc_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ------------------------------------------------------------------ bf16 */

/* bf16 -> real number: a bf16 is the upper half of an IEEE binary32. */
double orc_bf16_to_double(uint16_t b)
{
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* real number -> nearest bf16, ties to the even significand.  bf16 has an
 * 8-bit significand (1 implicit + 7 stored) and binary32's exponent range, so
 * the spacing of representable values around x is 2^(e-7) with
 * e = max(floor(log2|x|), -126). */
uint16_t orc_bf16_from_double(double x)
{
    uint16_t sign = (uint16_t)(signbit(x) ? 0x8000u : 0u);
    if (isnan(x)) return (uint16_t)(sign | 0x7FC0u);
    double a = fabs(x);
    if (isinf(a)) return (uint16_t)(sign | 0x7F80u);
    if (a == 0.0) return sign;
    int e;
    (void)frexp(a, &e);          /* a = f * 2^e, f in [0.5, 1)  =>  floor(log2 a) = e - 1 */
    e -= 1;
    if (e < -126) e = -126;
    double ulp = ldexp(1.0, e - 7);
    double r = nearbyint(a / ulp) * ulp;   /* default rounding mode: to nearest, ties to even; a/ulp is exact */
    if (r >= ldexp(1.0, 128)) return (uint16_t)(sign | 0x7F80u);
    float f = (float)r;                    /* exact: r has at most 8 significant bits */
    uint32_t u;
    memcpy(&u, &f, sizeof u);
    return (uint16_t)(sign | (uint16_t)(u >> 16));
}

/* ------------------------------------------------------- n-gram helpers */

/* The trailing n-gram ending at position t of sequence b: x[b][t-n+1 .. t].
 * Returns 0 when it would start before the sequence or contains a padding id. */
static int trailing_ngram(const int32_t *tokens, int32_t T, int32_t b, int32_t t,
                          int32_t n, int32_t vocab, int32_t gram[ORC_MAX_ORDERS])
{
    if (t - n + 1 < 0) return 0;
    for (int32_t k = 0; k < n; ++k) {
        int32_t x = tokens[(int64_t)b * T + (t - n + 1 + k)];
        if (x < 0 || x >= vocab) return 0;
        gram[k] = x;
    }
    return 1;
}

static int phrase_equals(const int32_t *phrase_tokens, const uint8_t *phrase_len,
                         int64_t i, const int32_t *gram, int32_t n)
{
    if ((int32_t)phrase_len[i] != n) return 0;
    for (int32_t k = 0; k < n; ++k)
        if (phrase_tokens[i * 4 + k] != gram[k]) return 0;
    return 1;
}

/* ------------------------------------------------ exact match, matcher O1 */

/* Brute force: for every query position and every order scan all N phrases.
 * match[q][oi] = phrase id whose tuple equals the trailing orders[oi]-gram, or -1.
 * [Sec. 4.2: the tokenised form tau_i is what inference-time matching uses.] */
void orc_match_brute(int64_t N, const int32_t *phrase_tokens, const uint8_t *phrase_len,
                     const int32_t *tokens, int32_t B, int32_t T, int32_t q_start,
                     int32_t vocab, int32_t n_orders, const int32_t *orders,
                     int64_t *match)
{
    int32_t Tq = T - q_start;
    for (int32_t b = 0; b < B; ++b)
        for (int32_t t = q_start; t < T; ++t) {
            int64_t q = (int64_t)b * Tq + (t - q_start);
            for (int32_t oi = 0; oi < n_orders; ++oi) {
                int32_t gram[ORC_MAX_ORDERS];
                int64_t found = -1;
                if (trailing_ngram(tokens, T, b, t, orders[oi], vocab, gram))
                    for (int64_t i = 0; i < N; ++i)
                        if (phrase_equals(phrase_tokens, phrase_len, i, gram, orders[oi])) {
                            found = i;
                            break;
                        }
                match[q * n_orders + oi] = found;
            }
        }
}

/* ------------------------------------------------ exact match, matcher O2 */

/* Total order on (length, tokens): shorter first, then lexicographic. */
static int tuple_cmp(int32_t na, const int32_t *a, int32_t nb, const int32_t *b)
{
    if (na != nb) return na < nb ? -1 : 1;
    for (int32_t k = 0; k < na; ++k)
        if (a[k] != b[k]) return a[k] < b[k] ? -1 : 1;
    return 0;
}

typedef struct {
    const int32_t *phrase_tokens;
    const uint8_t *phrase_len;
} sort_ctx;

static int perm_cmp(const void *pa, const void *pb, void *vctx)
{
    const sort_ctx *c = (const sort_ctx *)vctx;
    int64_t a = *(const int64_t *)pa, b = *(const int64_t *)pb;
    return tuple_cmp(c->phrase_len[a], c->phrase_tokens + a * 4,
                     c->phrase_len[b], c->phrase_tokens + b * 4);
}

/* perm[0..N) <- phrase ids in ascending (length, tokens) order.
 * Returns the number of adjacent equal tuples (0 for a valid table). */
int64_t orc_sort_phrases(int64_t N, const int32_t *phrase_tokens, const uint8_t *phrase_len,
                         int64_t *perm)
{
    sort_ctx c = { phrase_tokens, phrase_len };
    for (int64_t i = 0; i < N; ++i) perm[i] = i;
    qsort_r(perm, (size_t)N, sizeof(int64_t), perm_cmp, &c);
    int64_t dup = 0;
    for (int64_t i = 1; i < N; ++i)
        if (perm_cmp(&perm[i - 1], &perm[i], &c) == 0) ++dup;
    return dup;
}

/* Sorted search: binary search (lower bound) for the trailing n-gram in the
 * sorted phrase order.  Same output contract as orc_match_brute. */
void orc_match_sorted(int64_t N, const int32_t *phrase_tokens, const uint8_t *phrase_len,
                      const int64_t *perm,
                      const int32_t *tokens, int32_t B, int32_t T, int32_t q_start,
                      int32_t vocab, int32_t n_orders, const int32_t *orders,
                      int64_t *match)
{
    int32_t Tq = T - q_start;
    int64_t Q = (int64_t)B * Tq;
#pragma omp parallel for schedule(static)
    for (int64_t q = 0; q < Q; ++q) {
        int32_t b = (int32_t)(q / Tq), t = (int32_t)(q % Tq) + q_start;
        for (int32_t oi = 0; oi < n_orders; ++oi) {
            int32_t gram[ORC_MAX_ORDERS];
            int64_t found = -1;
            if (trailing_ngram(tokens, T, b, t, orders[oi], vocab, gram)) {
                int64_t lo = 0, hi = N;            /* first position whose tuple is >= gram */
                while (lo < hi) {
                    int64_t mid = lo + (hi - lo) / 2;
                    int64_t i = perm[mid];
                    if (tuple_cmp(phrase_len[i], phrase_tokens + i * 4, orders[oi], gram) < 0)
                        lo = mid + 1;
                    else
                        hi = mid;
                }
                if (lo < N && phrase_equals(phrase_tokens, phrase_len, perm[lo], gram, orders[oi]))
                    found = perm[lo];
            }
            match[q * n_orders + oi] = found;
        }
    }
}

/* ------------------------------------- selection, tier walk, miss hand-off */

static uint8_t tier_flag(int32_t slot_state)
{
    if (slot_state >= 0) return 1;       /* value already in the GPU cache: usable now      */
    if (slot_state == -1) return 2;      /* in host DRAM: must be staged to the GPU first   */
    return 3;                            /* only on SSD: asynchronous read, insert on arrival */
}

/* From the per-order matches decide, for every query, which phrase(s) are
 * retained [Sec. 4.2: deterministic policy, longer phrases preferred; or all
 * matches retained] and walk the hierarchy for each [Sec. 4.3].
 *
 * LONGEST: outputs are [Q].  The retained phrase is the matched one of
 *          greatest order; orders are ascending, so it is the last match.
 * ALL:     outputs are [Q][n_orders], column oi <-> orders[oi].
 *
 * Every retained phrase that is not in the GPU tier is appended to the miss
 * list (query index, phrase id, tier flag 2 or 3) in ascending (q, order);
 * duplicates are kept.  Returns the miss count. */
int64_t orc_select(int32_t policy, int64_t Q, int32_t n_orders, const int64_t *match,
                   const int32_t *slot_state,
                   uint32_t *sel_phrase, int32_t *sel_slot, uint8_t *flags,
                   uint32_t *miss_q, uint32_t *miss_phrase, uint8_t *miss_tier)
{
    int64_t n_miss = 0;
    for (int64_t q = 0; q < Q; ++q) {
        if (policy == ORC_POLICY_LONGEST) {
            int64_t best = -1;
            for (int32_t oi = 0; oi < n_orders; ++oi)
                if (match[q * n_orders + oi] >= 0) best = match[q * n_orders + oi];
            if (best < 0) {
                sel_phrase[q] = ORC_ABSENT_PHRASE; sel_slot[q] = -3; flags[q] = 0;
                continue;
            }
            int32_t s = slot_state[best];
            sel_phrase[q] = (uint32_t)best;
            sel_slot[q] = s >= 0 ? s : (s == -1 ? -1 : -2);
            flags[q] = tier_flag(s);
            if (flags[q] != 1) {
                miss_q[n_miss] = (uint32_t)q; miss_phrase[n_miss] = (uint32_t)best;
                miss_tier[n_miss] = flags[q]; ++n_miss;
            }
        } else {
            for (int32_t oi = 0; oi < n_orders; ++oi) {
                int64_t k = q * n_orders + oi, i = match[k];
                if (i < 0) {
                    sel_phrase[k] = ORC_ABSENT_PHRASE; sel_slot[k] = -3; flags[k] = 0;
                    continue;
                }
                int32_t s = slot_state[i];
                sel_phrase[k] = (uint32_t)i;
                sel_slot[k] = s >= 0 ? s : (s == -1 ? -1 : -2);
                flags[k] = tier_flag(s);
                if (flags[k] != 1) {
                    miss_q[n_miss] = (uint32_t)q; miss_phrase[n_miss] = (uint32_t)i;
                    miss_tier[n_miss] = flags[k]; ++n_miss;
                }
            }
        }
    }
    return n_miss;
}

/* ------------------------------------------------ aggregation + injection */

static double hidden_at(const void *h, int32_t hidden_dtype, int64_t idx)
{
    if (hidden_dtype == ORC_HIDDEN_F32) return (double)((const float *)h)[idx];
    return orc_bf16_to_double(((const uint16_t *)h)[idx]);
}

/* h'_t = h_t + g_t * m_t  [Sec. 2.2 injection eq.] for every query whose
 * retained phrase(s) include a GPU-resident one; every other query keeps h_t
 * unchanged.
 *
 *   m_t  LONGEST: the row of the selected phrase.
 *        ALL:     sum over the matched phrases that are GPU-resident of
 *                 alpha_i * row_i, alpha_i = n_i / (sum of n_j over ALL matched
 *                 phrases of this query, resident or not)  [Sec. 4.2 e_phi eq.;
 *                 weights by phrase length, one of the choices Sec. 4.2 allows].
 *   g_t  CONST:   lambda.
 *        COSINE:  lambda * sigmoid( <h,m> / sqrt(<h,h><m,m> + 1e-12) ).
 *
 * sel_slot / flags are orc_select's outputs for the same policy.  out_exact
 * (double [Q][d]) receives the unrounded value; out_rounded receives it in the
 * hidden dtype (bf16 bits or float), rounded to nearest even.  For untouched
 * queries out_rounded is a bitwise copy of h.  Either output may be NULL. */
void orc_inject(int32_t policy, int32_t gate, double lambda, int64_t Q, int32_t d,
                int32_t n_orders, const int32_t *orders,
                const int32_t *sel_slot, const uint8_t *flags,
                const uint16_t *rows, const void *h, int32_t hidden_dtype,
                double *out_exact, void *out_rounded)
{
#pragma omp parallel
    {
        double *m = (double *)malloc(sizeof(double) * (size_t)d);
#pragma omp for schedule(static)
        for (int64_t q = 0; q < Q; ++q) {
            int have_m = 0;
            if (policy == ORC_POLICY_LONGEST) {
                if (flags[q] == 1) {
                    have_m = 1;
                    for (int32_t j = 0; j < d; ++j)
                        m[j] = orc_bf16_to_double(rows[(int64_t)sel_slot[q] * d + j]);
                }
            } else {
                double n_sum = 0.0;
                for (int32_t oi = 0; oi < n_orders; ++oi)
                    if (flags[q * n_orders + oi] != 0) n_sum += (double)orders[oi];
                for (int32_t j = 0; j < d; ++j) m[j] = 0.0;
                for (int32_t oi = 0; oi < n_orders; ++oi) {
                    if (flags[q * n_orders + oi] != 1) continue;
                    have_m = 1;
                    double alpha = (double)orders[oi] / n_sum;
                    const uint16_t *row = rows + (int64_t)sel_slot[q * n_orders + oi] * d;
                    for (int32_t j = 0; j < d; ++j) m[j] += alpha * orc_bf16_to_double(row[j]);
                }
            }
            double g = lambda;
            if (have_m && gate == ORC_GATE_COSINE) {
                double s = 0.0, a = 0.0, c = 0.0;
                for (int32_t j = 0; j < d; ++j) {
                    double hj = hidden_at(h, hidden_dtype, q * d + j);
                    s += hj * m[j]; a += hj * hj; c += m[j] * m[j];
                }
                g = lambda / (1.0 + exp(-s / sqrt(a * c + 1e-12)));
            }
            for (int32_t j = 0; j < d; ++j) {
                int64_t idx = q * d + j;
                double hj = hidden_at(h, hidden_dtype, idx);
                double v = have_m ? hj + g * m[j] : hj;
                if (out_exact) out_exact[idx] = v;
                if (!out_rounded) continue;
                if (hidden_dtype == ORC_HIDDEN_F32)
                    ((float *)out_rounded)[idx] = have_m ? (float)v : ((const float *)h)[idx];
                else
                    ((uint16_t *)out_rounded)[idx] =
                        have_m ? orc_bf16_from_double(v) : ((const uint16_t *)h)[idx];
            }
        }
        free(m);
    }
}

/* --------------------------------------------------- GPU-tier installation */

/* Insert n fetched entries into the GPU tier [Sec. 4.3].  Entry k = phrase
 * ids[k] with row src[k][0..d) goes to slot dst[k].  Preconditions (checked;
 * on violation nothing changes and the 1-based index of the first offending
 * check is returned as a negative number):
 *   -1 an id is not a phrase;       -2 a phrase is already GPU-resident;
 *   -3 a slot is outside [0, C);    -4 ids not pairwise distinct;
 *   -5 slots not pairwise distinct.
 * Effects, for k in order: the phrase that owned dst[k], if any, falls back to
 * the host-DRAM tier (eviction); rows[dst[k]] <- src[k]; the phrase becomes
 * GPU-resident at dst[k].  slot_owner int64 [C]: phrase id or -1.  Returns 0. */
int32_t orc_cache_install(int64_t N, int64_t C, int32_t d,
                          int32_t *slot_state, int64_t *slot_owner, uint16_t *rows,
                          int32_t n, const uint32_t *ids, const uint16_t *src, const int32_t *dst)
{
    for (int32_t k = 0; k < n; ++k) {
        if ((int64_t)ids[k] >= N) return -1;
        if (slot_state[ids[k]] >= 0) return -2;
        if (dst[k] < 0 || (int64_t)dst[k] >= C) return -3;
    }
    for (int32_t k = 0; k < n; ++k)
        for (int32_t l = 0; l < k; ++l) {
            if (ids[k] == ids[l]) return -4;
            if (dst[k] == dst[l]) return -5;
        }
    for (int32_t k = 0; k < n; ++k) {
        int64_t prev = slot_owner[dst[k]];
        if (prev >= 0) slot_state[prev] = -1;
        if (rows && src)
            memcpy(rows + (int64_t)dst[k] * d, src + (int64_t)k * d, sizeof(uint16_t) * (size_t)d);
        slot_state[ids[k]] = dst[k];
        slot_owner[dst[k]] = (int64_t)ids[k];
    }
    return 0;
}

/* The same insertion for a caller that cannot check its batch beforehand -- a prefetch loop that
 * stays on the device hands over whatever the candidate step produced [Sec. 4.4: candidates are
 * fetched and inserted while the model computes].  Entries that cannot be applied are skipped
 * instead of refusing the batch.  Whether entry k is applied is judged against the state BEFORE
 * the call:
 *   candidate[k]: ids[k] is a phrase, it was not GPU-resident, dst[k] is a slot, and no earlier
 *                 entry of the batch names the same phrase;
 *   applied[k]:   candidate[k], and no earlier candidate of the batch names the same slot.
 * The applied entries then take effect in order, exactly as above.  Returns their number;
 * applied (uint8 [n]) receives the flags. */
int32_t orc_cache_install_lenient(int64_t N, int64_t C, int32_t d,
                                  int32_t *slot_state, int64_t *slot_owner, uint16_t *rows,
                                  int32_t n, const uint32_t *ids, const uint16_t *src, const int32_t *dst,
                                  uint8_t *applied)
{
    uint8_t *cand = (uint8_t *)malloc((size_t)(n > 0 ? n : 1));
    for (int32_t k = 0; k < n; ++k) {
        int ok = (int64_t)ids[k] < N && slot_state[ids[k]] < 0 && dst[k] >= 0 && (int64_t)dst[k] < C;
        for (int32_t l = 0; ok && l < k; ++l)
            if (ids[l] == ids[k]) ok = 0;
        cand[k] = (uint8_t)ok;
    }
    int32_t count = 0;
    for (int32_t k = 0; k < n; ++k) {
        int ok = cand[k];
        for (int32_t l = 0; ok && l < k; ++l)
            if (cand[l] && dst[l] == dst[k]) ok = 0;
        applied[k] = (uint8_t)ok;
        count += ok;
    }
    for (int32_t k = 0; k < n; ++k) {
        if (!applied[k]) continue;
        int64_t prev = slot_owner[dst[k]];
        if (prev >= 0) slot_state[prev] = -1;
        if (rows && src)
            memcpy(rows + (int64_t)dst[k] * d, src + (int64_t)k * d, sizeof(uint16_t) * (size_t)d);
        slot_state[ids[k]] = dst[k];
        slot_owner[dst[k]] = (int64_t)ids[k];
    }
    free(cand);
    return count;
}

/* ------------------------------------------------ GPU-tier retention ranking */

/* The paper ranks cached entries by signals -- access frequency and recency first among them --
 * and prints no formula [Sec. 4.3, cache policy].  PARITY UNPINNED BY THE PAPER: the reading below
 * is this build's, pinned by its special cases (pure LRU, pure LFU, free slots first).
 *
 * State per GPU-tier slot: freq = number of injections served from the slot since its row was
 * installed, last = epoch of the most recent one.  The epoch counts lookup calls.  A lookup at epoch
 * e adds 1 to freq and sets last = e for every entry it injects from the GPU tier (flag 1); an
 * install at epoch e sets freq = 1, last = e (the row counts as used once, now).
 *
 * Retention key of a slot at epoch `now` (larger = more worth keeping), all in unsigned 32-bit:
 *     age     = now - last
 *     decayed = freq >> min(31, age / half_life)        (half_life <= 0: no decay)
 *     key     = min(decayed, 65535) << 16  |  (65535 - min(age, 65535))
 * i.e. frequency halved once per half_life idle epochs, ties broken by recency.  A slot without an
 * owner has key 0.  Victims are the n slots of smallest (key, slot), in that order. */
void orc_cache_touch(int64_t n_ent, const uint8_t *flags, const int32_t *sel_slot, uint32_t epoch,
                     uint32_t *freq, uint32_t *last)
{
    for (int64_t e = 0; e < n_ent; ++e)
        if (flags[e] == 1) {
            freq[sel_slot[e]] += 1u;
            last[sel_slot[e]] = epoch;
        }
}

void orc_cache_installed(int32_t n, const int32_t *dst_slots, uint32_t epoch, uint32_t *freq, uint32_t *last)
{
    for (int32_t k = 0; k < n; ++k) {
        freq[dst_slots[k]] = 1u;
        last[dst_slots[k]] = epoch;
    }
}

uint32_t orc_retention_key(uint32_t freq, uint32_t last, uint32_t now, int32_t half_life)
{
    const uint32_t age = now - last;
    uint32_t shift = 0;
    if (half_life > 0) {
        shift = age / (uint32_t)half_life;
        if (shift > 31u) shift = 31u;
    }
    uint32_t decayed = freq >> shift;
    if (decayed > 65535u) decayed = 65535u;
    return (decayed << 16) | (65535u - (age > 65535u ? 65535u : age));
}

typedef struct { uint32_t key; int32_t slot; } orc_slot_rank;

static int slot_rank_cmp(const void *pa, const void *pb)
{
    const orc_slot_rank *a = (const orc_slot_rank *)pa, *b = (const orc_slot_rank *)pb;
    if (a->key != b->key) return a->key < b->key ? -1 : 1;
    return a->slot < b->slot ? -1 : (a->slot > b->slot ? 1 : 0);
}

/* slot_owner[s] < 0: slot s is free.  Writes min(n, C) slots (and their keys) and returns that count. */
int64_t orc_cache_victims(int64_t C, const int64_t *slot_owner, const uint32_t *freq, const uint32_t *last,
                          uint32_t now, int32_t half_life, int64_t n, int32_t *out_slots, uint32_t *out_keys)
{
    orc_slot_rank *r = (orc_slot_rank *)malloc((size_t)(C > 0 ? C : 1) * sizeof *r);
    for (int64_t s = 0; s < C; ++s) {
        r[s].slot = (int32_t)s;
        r[s].key = slot_owner[s] < 0 ? 0u : orc_retention_key(freq[s], last[s], now, half_life);
    }
    qsort(r, (size_t)C, sizeof *r, slot_rank_cmp);
    const int64_t take = n < C ? n : C;
    for (int64_t k = 0; k < take; ++k) {
        out_slots[k] = r[k].slot;
        if (out_keys) out_keys[k] = r[k].key;
    }
    free(r);
    return take;
}

/* ------------------------------------------- prefetch candidates + priority */

/* Early-exit guided prefetching, the part after the top-K tokens are known [Sec. 4.4]: each
 * predicted next token cand[b][k] (probability prob[b][k]) is combined with the recent history of
 * its sequence into the n-grams it would complete -- (history[b][H-n+1 .. H-1], cand[b][k]) for
 * every configured order n -- and looked up in the phrase table [Sec. 4.4, candidate set Q_t].  A
 * phrase that is found and is not in the GPU tier is a prefetch candidate with priority
 *     s = p * r * c          [Sec. 4.4, priority score]
 * p = prob[b][k], r = usefulness[phrase] (1 if usefulness is NULL), c = benefit of fetching it
 * from its tier (benefit_host or benefit_ssd; entries already in the GPU tier have no benefit and
 * are not candidates).  The product is taken in single precision, left to right, because the
 * ranking is decided by it and the GPU ranks in single precision.  Candidates with s <= 0 are
 * dropped.  The `budget` candidates of highest priority are returned in descending priority; equal
 * priorities keep ascending (b, k, order).  Duplicates (one phrase reached from several tokens)
 * are kept.
 *
 * out_src = b*K + k.  Returns the number of candidates before the budget cut; the first
 * min(budget, that number) output entries are valid.  Uses the sorted phrase order `perm`. */
typedef struct { float score; uint32_t idx, phrase, src; uint8_t tier; } orc_cand;

static int cand_cmp(const void *pa, const void *pb)
{
    const orc_cand *a = (const orc_cand *)pa, *b = (const orc_cand *)pb;
    if (a->score != b->score) return a->score > b->score ? -1 : 1;
    return a->idx < b->idx ? -1 : (a->idx > b->idx ? 1 : 0);
}

int64_t orc_prefetch_candidates(int64_t N, const int32_t *phrase_tokens, const uint8_t *phrase_len,
                                const int64_t *perm, const int32_t *slot_state,
                                const int32_t *history, int32_t B, int32_t H,
                                const int32_t *cand, const float *prob, int32_t K,
                                int32_t vocab, int32_t n_orders, const int32_t *orders,
                                const float *usefulness, float benefit_host, float benefit_ssd, int32_t budget,
                                uint32_t *out_phrase, uint8_t *out_tier, float *out_score, uint32_t *out_src)
{
    int64_t cap = (int64_t)B * K * n_orders, n = 0;
    orc_cand *list = (orc_cand *)malloc(sizeof(orc_cand) * (size_t)(cap > 0 ? cap : 1));
    for (int32_t b = 0; b < B; ++b)
        for (int32_t k = 0; k < K; ++k)
            for (int32_t oi = 0; oi < n_orders; ++oi) {
                int32_t no = orders[oi], gram[ORC_MAX_ORDERS], ok = no - 1 <= H;
                for (int32_t j = 0; ok && j < no - 1; ++j) {
                    gram[j] = history[(int64_t)b * H + (H - (no - 1) + j)];
                    if (gram[j] < 0 || gram[j] >= vocab) ok = 0;
                }
                if (!ok) continue;
                gram[no - 1] = cand[(int64_t)b * K + k];
                if (gram[no - 1] < 0 || gram[no - 1] >= vocab) continue;
                int64_t lo = 0, hi = N;
                while (lo < hi) {
                    int64_t mid = lo + (hi - lo) / 2, i = perm[mid];
                    if (tuple_cmp(phrase_len[i], phrase_tokens + i * 4, no, gram) < 0) lo = mid + 1; else hi = mid;
                }
                if (lo >= N || !phrase_equals(phrase_tokens, phrase_len, perm[lo], gram, no)) continue;
                int64_t id = perm[lo];
                if (slot_state[id] >= 0) continue;                 /* already in the GPU tier */
                float c = slot_state[id] == -1 ? benefit_host : benefit_ssd;
                float r = usefulness ? usefulness[id] : 1.0f;
                float pr = prob[(int64_t)b * K + k] * r;
                float s = pr * c;
                if (!(s > 0.0f)) continue;
                list[n].score = s; list[n].idx = (uint32_t)(((int64_t)b * K + k) * n_orders + oi);
                list[n].phrase = (uint32_t)id; list[n].src = (uint32_t)((int64_t)b * K + k);
                list[n].tier = (uint8_t)(slot_state[id] == -1 ? 2 : 3);
                ++n;
            }
    qsort(list, (size_t)n, sizeof(orc_cand), cand_cmp);
    for (int64_t i = 0; i < n && i < budget; ++i) {
        out_phrase[i] = list[i].phrase; out_tier[i] = list[i].tier;
        out_score[i] = list[i].score; out_src[i] = list[i].src;
    }
    free(list);
    return n;
}

/* ------------------------------------------------ early-exit prefetch head */

/* The auxiliary head at layer L-r turns the intermediate hidden state of every sequence into an
 * approximate next-token distribution
 *     p_early = softmax(W_pref h)            [Sec. 4.4, p_early equation]
 * and keeps its K most likely tokens
 *     T_early = TopK(p_early)                [Sec. 4.4, T_early equation].
 * W_pref is [V][d], h is [B][d], both bf16 bit patterns; everything else in double.
 *
 * orc_head_logits: z[b][v] = sum_j W[v][j] * h[b][j], summed in ascending j. */
void orc_head_logits(int32_t V, int32_t d, int32_t B, const uint16_t *W, const uint16_t *h, double *z)
{
#pragma omp parallel for schedule(static)
    for (int64_t v = 0; v < V; ++v)
        for (int32_t b = 0; b < B; ++b) {
            double acc = 0.0;
            for (int32_t j = 0; j < d; ++j)
                acc += orc_bf16_to_double(W[(size_t)v * d + j]) * orc_bf16_to_double(h[(size_t)b * d + j]);
            z[(size_t)b * V + v] = acc;
        }
}

/* orc_head_topk: for every row of z the softmax over all V entries (with the usual subtraction of
 * the row maximum, which cancels) and the K entries of largest probability, in descending
 * probability; equal logits keep ascending token id.  tokens [B][K], prob [B][K]; lse[b] receives
 * log(sum_v exp(z[b][v])) when lse is not NULL.  K <= V. */
typedef struct { double z; int32_t v; } orc_logit;

static int logit_cmp(const void *pa, const void *pb)
{
    const orc_logit *a = (const orc_logit *)pa, *b = (const orc_logit *)pb;
    if (a->z != b->z) return a->z > b->z ? -1 : 1;
    return a->v < b->v ? -1 : (a->v > b->v ? 1 : 0);
}

void orc_head_topk(int32_t V, int32_t B, int32_t K, const double *z, int32_t *tokens, double *prob, double *lse)
{
#pragma omp parallel for schedule(static)
    for (int32_t b = 0; b < B; ++b) {
        const double *row = z + (size_t)b * V;
        orc_logit *r = (orc_logit *)malloc((size_t)V * sizeof *r);
        double top = row[0];
        for (int32_t v = 0; v < V; ++v) {
            r[v].z = row[v];
            r[v].v = v;
            if (row[v] > top) top = row[v];
        }
        double sum = 0.0;
        for (int32_t v = 0; v < V; ++v) sum += exp(row[v] - top);
        qsort(r, (size_t)V, sizeof *r, logit_cmp);
        for (int32_t k = 0; k < K; ++k) {
            tokens[(size_t)b * K + k] = r[k].v;
            prob[(size_t)b * K + k] = exp(r[k].z - top) / sum;
        }
        if (lse) lse[b] = top + log(sum);
        free(r);
    }
}

/* ------------------------------------------------------------------------------------------------
 * N-gram extraction with a frequency threshold [Sec. 4.2 construction pipeline: candidate phrases
 * are multi-token expressions such as bigrams and trigrams, selected by a frequency threshold;
 * Sec. 5.3: this tokenizer-level n-gram extraction is the dominant offline cost].
 *
 * corpus   tokens int32 [L]; an id outside [0, vocab) separates documents: no window contains one.
 * window   for a configured order n and an end position t >= n - 1 whose n ids x_{t-n+1} .. x_t are
 *          all valid, that tuple occurs once at t.
 * count(tuple) = number of its occurrences, first(tuple) = its smallest end position.
 *
 * Result: the tuples with count >= min_count, in ascending (first, n) order -- the order in which a
 * reader of the corpus meets them.  Returns how many there are; writes the first `cap` of them
 * (out_tokens [cap][4] padded with -1, out_len, out_count).  distinct[oi] = number of different
 * tuples of order orders[oi].  hist (length hist_bins, may be NULL): hist[c] = number of different
 * tuples, all orders together, that occur exactly c times, the last bin collecting every c >=
 * hist_bins - 1.
 *
 * Method: the definition.  Every window becomes a record; records are sorted by (n, tuple, t), so that
 * the occurrences of one tuple are adjacent and its first one leads; the survivors are sorted by
 * (first, n). */
typedef struct { int32_t n, tok[ORC_MAX_ORDERS]; int64_t t; uint32_t count; } orc_window;

static int window_cmp(const void *pa, const void *pb)
{
    const orc_window *a = (const orc_window *)pa, *b = (const orc_window *)pb;
    if (a->n != b->n) return a->n < b->n ? -1 : 1;
    for (int j = 0; j < ORC_MAX_ORDERS; ++j)
        if (a->tok[j] != b->tok[j]) return a->tok[j] < b->tok[j] ? -1 : 1;
    return a->t < b->t ? -1 : (a->t > b->t ? 1 : 0);
}

static int first_cmp(const void *pa, const void *pb)
{
    const orc_window *a = (const orc_window *)pa, *b = (const orc_window *)pb;
    if (a->t != b->t) return a->t < b->t ? -1 : 1;
    return a->n < b->n ? -1 : (a->n > b->n ? 1 : 0);
}

int64_t orc_mine_ngrams(int64_t L, const int32_t *tokens, int32_t vocab, int32_t n_orders, const int32_t *orders,
                        uint32_t min_count, int64_t cap, int32_t *out_tokens, uint8_t *out_len, uint32_t *out_count,
                        int64_t *distinct, int32_t hist_bins, int64_t *hist)
{
    orc_window *w = (orc_window *)malloc((size_t)(L * n_orders + 1) * sizeof *w);
    int64_t n_w = 0;
    for (int64_t t = 0; t < L; ++t)
        for (int32_t oi = 0; oi < n_orders; ++oi) {
            const int32_t n = orders[oi];
            if (t < n - 1) continue;
            int valid = 1;
            for (int32_t j = 0; j < n; ++j) {
                const int32_t x = tokens[t - n + 1 + j];
                if (x < 0 || x >= vocab) valid = 0;
            }
            if (!valid) continue;
            w[n_w].n = n;
            for (int32_t j = 0; j < ORC_MAX_ORDERS; ++j) w[n_w].tok[j] = j < n ? tokens[t - n + 1 + j] : -1;
            w[n_w].t = t;
            w[n_w].count = 0;
            ++n_w;
        }
    qsort(w, (size_t)n_w, sizeof *w, window_cmp);
    for (int32_t oi = 0; oi < n_orders; ++oi) distinct[oi] = 0;
    if (hist) for (int32_t c = 0; c < hist_bins; ++c) hist[c] = 0;
    int64_t n_keep = 0;                         /* survivors are moved to the front of w */
    for (int64_t i = 0; i < n_w;) {
        int64_t j = i + 1;
        while (j < n_w && w[j].n == w[i].n && memcmp(w[j].tok, w[i].tok, sizeof w[i].tok) == 0) ++j;
        const int64_t count = j - i;            /* w[i] is the first occurrence: smallest t of the run */
        for (int32_t oi = 0; oi < n_orders; ++oi) if (orders[oi] == w[i].n) ++distinct[oi];
        if (hist) ++hist[count < hist_bins - 1 ? count : hist_bins - 1];
        if (count >= (int64_t)min_count) {
            w[n_keep] = w[i];
            w[n_keep].count = (uint32_t)count;
            ++n_keep;
        }
        i = j;
    }
    qsort(w, (size_t)n_keep, sizeof *w, first_cmp);
    for (int64_t i = 0; i < n_keep && i < cap; ++i) {
        for (int32_t j = 0; j < ORC_MAX_ORDERS; ++j) out_tokens[i * ORC_MAX_ORDERS + j] = w[i].tok[j];
        out_len[i] = (uint8_t)w[i].n;
        out_count[i] = w[i].count;
    }
    free(w);
    return n_keep;
}

/* orc_count_tuple: occurrences of ONE tuple of n ids in the corpus, by the definition above (a scan over
 * all end positions); *first receives the smallest end position, -1 if there is none.  For spot checks
 * on corpora that orc_mine_ngrams would take too long to sort. */
int64_t orc_count_tuple(int64_t L, const int32_t *tokens, int32_t n, const int32_t *tuple, int64_t *first)
{
    int64_t count = 0;
    *first = -1;
    for (int64_t t = n - 1; t < L; ++t) {
        int same = 1;
        for (int32_t j = 0; j < n; ++j)
            if (tokens[t - n + 1 + j] != tuple[j]) same = 0;
        if (same) {
            if (count == 0) *first = t;
            ++count;
        }
    }
    return count;
}

/* ------------------------------------------------------------------------------------------------
 * Initial residency from corpus counts [Sec. 4.3: the GPU tier is reserved for the most frequently
 * accessed entries, DRAM holds warm entries, SSD absorbs the long tail].
 *
 * The G = min(gpu_slots, N) phrases of largest count start in the GPU tier; among equal counts the
 * smaller id goes first.  GPU-tier slots are handed out in id order: the chosen phrase with the k-th
 * smallest id gets slot k.  Of the others, a count >= host_min_count means host DRAM (-1), a smaller
 * one SSD (-2).  tiers[0..2] receive the number of phrases per tier (GPU, host, SSD). */
typedef struct { uint32_t count; int64_t id; } orc_ranked;

static int ranked_cmp(const void *pa, const void *pb)
{
    const orc_ranked *a = (const orc_ranked *)pa, *b = (const orc_ranked *)pb;
    if (a->count != b->count) return a->count > b->count ? -1 : 1;
    return a->id < b->id ? -1 : (a->id > b->id ? 1 : 0);
}

void orc_assign_residency(int64_t N, const uint32_t *count, int64_t gpu_slots, uint32_t host_min_count,
                          int32_t *init_slot, int64_t *tiers)
{
    orc_ranked *r = (orc_ranked *)malloc((size_t)(N + 1) * sizeof *r);
    for (int64_t i = 0; i < N; ++i) { r[i].count = count[i]; r[i].id = i; }
    qsort(r, (size_t)N, sizeof *r, ranked_cmp);
    const int64_t G = gpu_slots < N ? gpu_slots : N;
    tiers[0] = tiers[1] = tiers[2] = 0;
    for (int64_t i = 0; i < N; ++i) init_slot[i] = count[i] >= host_min_count ? -1 : -2;
    for (int64_t k = 0; k < G; ++k) init_slot[r[k].id] = 0;           /* chosen; numbered below */
    int32_t next = 0;
    for (int64_t i = 0; i < N; ++i) {
        if (init_slot[i] == 0) init_slot[i] = next++;
        ++tiers[init_slot[i] >= 0 ? 0 : (init_slot[i] == -1 ? 1 : 2)];
    }
    free(r);
}
