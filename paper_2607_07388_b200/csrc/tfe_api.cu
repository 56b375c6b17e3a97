// Host side of libtfe.so: the C ABI declared in include/tfe.h.
//
// The context owns the device index, the per-phrase metadata the kernels need
// (index position of every phrase, token tuples of hashed orders, owner of every
// GPU-tier slot), the miss-list buffers, and a host mirror of the residency state
// used to validate arguments before anything is launched.
#include <algorithm>
#include <climits>
#include <cmath>
#include <cstdint>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <new>
#include <string>
#include <vector>

#include "../../include/tfe.h"
#include "tfe_kernels.cuh"

namespace {

thread_local std::string g_cuda_error;

bool cuda_failed(cudaError_t e, const char *what)
{
    if (e == cudaSuccess) return false;
    g_cuda_error = std::string(what) + ": " + cudaGetErrorString(e);
    (void)cudaGetLastError();
    return true;
}
#define CU(call)                                                       \
    do {                                                               \
        if (cuda_failed((call), #call)) return TFE_ERR_CUDA;           \
    } while (0)

// Launch with programmatic stream serialisation: the launch is set up while the kernel before it on the
// stream drains.  Only for kernels that call tfe_grid_dependency_sync() before their first global access.
template <class... KArgs, class... Args>
cudaError_t launch_overlapped(void (*kernel)(KArgs...), dim3 grid, dim3 block, cudaStream_t stream, Args... args)
{
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = 0; cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

constexpr uint32_t kNoOwner = 0xFFFFFFFFu;
constexpr int kDefaultMaxKicks = 2000;
constexpr int kVarSlots = 24;

}  // namespace

struct tfe_ctx {
    tfe_config cfg{};
    int device = 0;
    int sm_count = 0;
    int tok_bits = 0;
    bool any_hashed = false;
    uint64_t n_buckets = 0;
    int row_vecs = 0;                       // 16-byte vectors per GPU-tier row

    void *d_arena = nullptr;                // device build: index, positions, owners, counters (and tuples) are one allocation
    ulonglong2 *d_index = nullptr;
    int4 *d_phrase_tokens = nullptr;        // only when an order is hashed
    uint32_t *d_phrase_pos = nullptr;
    uint32_t *d_slot_owner = nullptr;
    uint4 *gpu_rows = nullptr;              // caller-owned

    std::vector<int32_t> h_slot;            // residency mirror
    std::vector<uint32_t> h_owner;

    int64_t ent_cap = 0;                    // capacity (entries) of the five buffers below
    unsigned long long *d_scr_rec = nullptr;        // one result record per (query, order column) of the last lookup
    uint32_t *d_miss_q = nullptr, *d_miss_phrase = nullptr;
    uint8_t *d_miss_tier = nullptr;
    uint32_t *d_counters = nullptr;         // TFE_CTR_WORDS words of launch state
    int occ[kVarSlots] = {0};
    // resident blocks per SM of each kernel variant

    int64_t last_entries = -1;              // Q*cols of the most recent lookup (-1: none yet)
    int last_grid = 0, last_block = 0, last_qb = 0;
    int qb_override = 0;                    // 0: choose per call

    // install staging
    uint32_t *d_inst_ids = nullptr;
    int32_t *d_inst_slots = nullptr;
    uint4 *d_inst_rows = nullptr;
    int32_t inst_cap = 0;

    // prefetch-candidate scratch
    unsigned long long *d_pf_keys = nullptr;
    uint32_t *d_pf_phrase = nullptr;
    uint8_t *d_pf_tier = nullptr;
    uint32_t *d_pf_counter = nullptr;
    int64_t pf_cap = 0;

    // retention ranking (tfe_cache_policy_enable): per-slot {freq, last}, the lookup count, and
    // the victim selection's work space
    uint2 *d_slot_stats = nullptr;
    uint32_t *d_epoch = nullptr;
    uint32_t *d_vs_keys = nullptr;
    TfeVictimState *d_vs_state = nullptr;
    unsigned long long *d_vs_list = nullptr, *d_vs_fin = nullptr;
    int32_t *d_vs_slots = nullptr;
    int vs_grid_max = 0;                    // blocks of the selection kernel the device holds at once
    int32_t vs_list_cap = 0, vs_final_cap = 0, vs_samples = 0;     // 0: the defaults (tfe_cache_select_tuning)

    bool mirror_ready = true;               // h_slot / h_owner filled (a device build fills them on first use)
    bool device_installs = false;           // tfe_cache_install_device was used: replays of a captured call change the
                                            // residency without the host seeing it, so the mirror is never trusted again

    // tfe_cache_install_device: stamps per phrase and per slot, the call counter, the applied count
    uint32_t *d_phrase_stamp = nullptr, *d_slot_stamp = nullptr, *d_inst_count = nullptr;
    uint8_t *d_inst_flags = nullptr;        // which entries of the device-side installation in flight are applied

    // host-buffer variant staging
    int32_t *d_h_tokens = nullptr;
    void *d_h_hidden = nullptr, *d_h_out = nullptr;
    uint32_t *d_h_phrase = nullptr;
    int32_t *d_h_slot = nullptr;
    uint8_t *d_h_flag = nullptr;
    int64_t hb_tok_cap = 0, hb_q_cap = 0, hb_ent_cap = 0;
    // copy streams and events of the host-buffer variant's pipeline (created on its first call)
    enum { kPipeMaxChunks = 32 };
    cudaStream_t hb_in = nullptr, hb_out = nullptr;
    cudaEvent_t hb_ev_start = nullptr, hb_ev_done = nullptr;
    cudaEvent_t hb_ev_in[kPipeMaxChunks] = {}, hb_ev_k[kPipeMaxChunks] = {};
};

namespace {

typedef void (*lookup_kernel_t)(const TfeLookupParams);

// Kernel variants.  0..7: hidden dtype x policy x gate, the general kernel in fp32 arithmetic.
// 8..10: the LONGEST / CONST kernel -- bf16 hidden in fp32 arithmetic, bf16 hidden with the
// packed bf16 fused multiply-add (lambda exactly a bf16 number), fp32 hidden.  11..13: the same
// three for a call issued in several launches over query ranges (variant + kVarRanged).  14..19: those six
// compiled for rows of several chunks (variant + kVarWide: half the registers in flight per lane, four blocks per SM).
// 20, 21: LONGEST / COSINE on rows one trip covers (bf16 / fp32 hidden): the LONGEST kernel with the gate.
enum { kVarLongest = 8, kVarLongestPacked = 9, kVarLongestF32 = 10, kVarRanged = 3, kVarWide = 6, kVarLongestCos = 20, kVarCount = 22 };
constexpr int kCosSteps = 128;         // 16-byte steps of h per row up to which kVarLongestCos applies ...
constexpr int64_t kCosMinQueries = 2048;   // ... and the call size from which

// The variants that can run a call in pieces and have a wide-row form.
inline bool is_longest_const(int variant) { return variant >= kVarLongest && variant < kVarLongestCos; }
constexpr int kWideSteps = 384;        // 16-byte steps of h per row from which the kVarWide variants are used

lookup_kernel_t pick_kernel(int variant)
{
    static const lookup_kernel_t table[kVarCount] = {
        tfe_lookup_inject_kernel<0, false, false, false>, tfe_lookup_inject_kernel<0, false, true, false>,
        tfe_lookup_inject_kernel<0, true, false, false>,  tfe_lookup_inject_kernel<0, true, true, false>,
        tfe_lookup_inject_kernel<1, false, false, false>, tfe_lookup_inject_kernel<1, false, true, false>,
        tfe_lookup_inject_kernel<1, true, false, false>,  tfe_lookup_inject_kernel<1, true, true, false>,
        tfe_lookup_inject_longest_kernel<0, false, false, 4>, tfe_lookup_inject_longest_kernel<0, true, false, 4>,
        tfe_lookup_inject_longest_kernel<1, false, false, 4>,
        tfe_lookup_inject_longest_kernel<0, false, true, 4>,  tfe_lookup_inject_longest_kernel<0, true, true, 4>,
        tfe_lookup_inject_longest_kernel<1, false, true, 4>,
        tfe_lookup_inject_longest_kernel<0, false, false, 2>, tfe_lookup_inject_longest_kernel<0, true, false, 2>,
        tfe_lookup_inject_longest_kernel<1, false, false, 2>,
        tfe_lookup_inject_longest_kernel<0, false, true, 2>,  tfe_lookup_inject_longest_kernel<0, true, true, 2>,
        tfe_lookup_inject_longest_kernel<1, false, true, 2>,
        tfe_lookup_inject_longest_kernel<0, false, false, 4, true>, tfe_lookup_inject_longest_kernel<1, false, false, 4, true>,
    };
    return table[variant];
}

// Queries per warp batch (1..8) for a call of Q queries on `warps` resident warps.  A split into r
// rounds of qb = ceil(Q / (warps*r)) queries gives the busiest warp r*qb queries; among the splits
// within 8 % of the least such load the largest batch wins (fewer probe phases per warp).  Small
// calls: one query per warp, the lowest latency.
int pick_batch(int64_t Q, int64_t warps, int max_qb = 8)
{
    if (Q <= warps) return 1;
    int64_t load[9];
    int64_t best = INT64_MAX;
    for (int qb = 1; qb <= max_qb; ++qb) {
        const int64_t r = (Q + warps * qb - 1) / (warps * qb);      // rounds needed with this batch size
        load[qb] = r * qb;
        best = std::min(best, load[qb]);
    }
    for (int qb = max_qb; qb >= 1; --qb)
        if (load[qb] * 100 <= best * 108) return qb;
    return 1;
}

// Most queries a warp batch of a variant holds: the LONGEST / CONST kernels give a query two lanes per order
// (at least four), the general kernels four.
int max_batch(const tfe_ctx *c, int variant)
{
    if (variant < kVarLongest) return 8;
    return std::min(8, 32 / std::max(4, 2 * c->cfg.n_orders));
}

// Launch geometry of a lookup over Qr queries: blocks and queries per warp round.
// General kernels: warps take batches of qb queries in a grid-strided order (pick_batch above).
// LONGEST / CONST kernels: warp w owns queries w, w + n_warps, ... (equal shares to within one query) and walks
// them in rounds of qb: as few rounds as the lanes allow, as even as the share allows.
void lookup_geometry(const tfe_ctx *c, int variant, int64_t Qr, int64_t *qb_out, int64_t *grid_out)
{
    const int64_t resident = (int64_t)c->sm_count * c->occ[variant];
    const int64_t cap = max_batch(c, variant);
    int64_t qb, grid;
    if (variant >= kVarLongest) {
        // batch size and grid as for the general kernels (few, full warps for small calls), then even shares
        const int64_t qb0 = c->qb_override ? std::min<int64_t>(c->qb_override, cap) : pick_batch(Qr, resident * TFE_WARPS_PER_BLOCK, (int)cap);
        const int64_t n_batches = (Qr + qb0 - 1) / qb0;
        grid = std::max<int64_t>(1, std::min<int64_t>(resident, (n_batches + TFE_WARPS_PER_BLOCK - 1) / TFE_WARPS_PER_BLOCK));
        const int64_t share = (Qr + grid * TFE_WARPS_PER_BLOCK - 1) / (grid * TFE_WARPS_PER_BLOCK);    // queries of the busiest warp
        const int64_t rounds = std::max<int64_t>(1, (share + qb0 - 1) / qb0);
        qb = std::max<int64_t>(1, (share + rounds - 1) / rounds);
    } else {
        qb = c->qb_override ? std::min<int64_t>(c->qb_override, cap) : pick_batch(Qr, resident * TFE_WARPS_PER_BLOCK, (int)cap);
        const int64_t n_batches = (Qr + qb - 1) / qb;
        grid = std::max<int64_t>(1, std::min<int64_t>(resident, (n_batches + TFE_WARPS_PER_BLOCK - 1) / TFE_WARPS_PER_BLOCK));
    }
    *qb_out = qb; *grid_out = grid;
}

TfeFastDiv make_fastdiv(uint32_t d)
{
    uint32_t s = 0;
    while ((1ull << s) < d) ++s;
    TfeFastDiv f;
    f.shr = 31 + s;
    f.mul = (uint32_t)((1ull << f.shr) / d + 1);
    return f;
}

void free_dev(void *p) { if (p) (void)cudaFree(p); }

// Resident blocks per SM of every lookup variant, asked of the runtime once per device and process.
cudaError_t lookup_occupancy(int device, int (&occ)[kVarSlots])
{
    constexpr int kMaxDevices = 64;
    static int cache[kMaxDevices][kVarSlots];
    static bool have[kMaxDevices];
    static std::mutex guard;
    std::lock_guard<std::mutex> lock(guard);
    const bool cached = device >= 0 && device < kMaxDevices;
    if (!cached || !have[device]) {
        int fresh[kVarSlots] = {};
        for (int v = 0; v < kVarCount; ++v) {
            int o = 0;
            const cudaError_t e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&o, pick_kernel(v), TFE_BLOCK_THREADS, 0);
            if (e != cudaSuccess) return e;
            fresh[v] = std::max(1, o);
        }
        if (!cached) { for (int v = 0; v < kVarSlots; ++v) occ[v] = fresh[v]; return cudaSuccess; }
        for (int v = 0; v < kVarSlots; ++v) cache[device][v] = fresh[v];
        have[device] = true;
    }
    for (int v = 0; v < kVarSlots; ++v) occ[v] = cache[device][v];
    return cudaSuccess;
}

tfe_status validate_config(const tfe_config *c)
{
    if (!c) return TFE_ERR_INVALID_ARG;
    if (c->d < 8 || c->d % 8 != 0) return TFE_ERR_INVALID_ARG;
    if (c->vocab < 1) return TFE_ERR_INVALID_ARG;
    if (c->n_orders < 1 || c->n_orders > 4) return TFE_ERR_INVALID_ARG;
    for (int i = 0; i < c->n_orders; ++i) {
        if (c->orders[i] < 1 || c->orders[i] > 4) return TFE_ERR_INVALID_ARG;
        if (i && c->orders[i] <= c->orders[i - 1]) return TFE_ERR_INVALID_ARG;
    }
    if (c->n_phrases < 0 || c->gpu_slots < 0) return TFE_ERR_INVALID_ARG;
    if (c->gpu_slots > 0x7FFFFFFFll) return TFE_ERR_INVALID_ARG;
    if (!(c->load_factor > 0.f && c->load_factor <= 1.f)) return TFE_ERR_INVALID_ARG;
    if (c->hidden_dtype != 0 && c->hidden_dtype != 1) return TFE_ERR_INVALID_ARG;
    if (c->max_kicks < 0) return TFE_ERR_INVALID_ARG;
    if (c->n_phrases > 0xFFFFFFFEll) return TFE_ERR_CAPACITY;
    return TFE_OK;
}

// Two-choice cuckoo placement of N keys into buckets of 4 slots (host, sequential, deterministic).
// slots[] receives {key, value}; pos[i] the slot index of phrase i.  A key goes to a free slot of
// either of its buckets; when both are full a resident key is moved to its other bucket, up to
// max_kicks moves per insertion.  Returns false if a key could not be placed.
struct HostSlot { uint64_t key, val; };

bool cuckoo_build(const std::vector<uint64_t> &keys, const int32_t *init_slot, uint64_t n_buckets, int max_kicks,
                  std::vector<HostSlot> &slots, std::vector<uint32_t> &pos)
{
    const size_t N = keys.size();
    slots.assign((size_t)n_buckets * TFE_SLOTS_PER_BUCKET, HostSlot{0, 0});
    pos.assign(std::max<size_t>(N, 1), 0);
    uint64_t rng = 0x853C49E6748FEA9Bull;
    auto try_place = [&](uint64_t bucket, uint64_t key, uint64_t val) -> bool {
        HostSlot *b = &slots[(size_t)bucket * TFE_SLOTS_PER_BUCKET];
        for (int s = 0; s < TFE_SLOTS_PER_BUCKET; ++s)
            if (b[s].key == 0) {
                b[s] = HostSlot{key, val};
                pos[(size_t)(val >> 32)] = (uint32_t)(bucket * TFE_SLOTS_PER_BUCKET + s);
                return true;
            }
        return false;
    };
    for (size_t i = 0; i < N; ++i) {
        uint64_t key = keys[i];
        uint64_t val = ((uint64_t)i << 32) | (uint32_t)init_slot[i];
        uint64_t avoid = UINT64_MAX;           // the bucket the key in hand was just taken from
        bool placed = false;
        for (int kick = 0; kick <= max_kicks; ++kick) {
            const uint64_t b1 = tfe_home_bucket_of(key, n_buckets);
            const uint64_t b2 = tfe_second_bucket_of(key, b1, n_buckets);
            if (try_place(b1, key, val) || try_place(b2, key, val)) { placed = true; break; }
            // both full: take a victim from the bucket we did not just come from
            const uint64_t from = b1 == avoid ? b2 : (b2 == avoid ? b1 : ((rng >> 40) & 1 ? b1 : b2));
            rng = rng * 6364136223846793005ull + 1442695040888963407ull;
            const int s = (int)((rng >> 33) % TFE_SLOTS_PER_BUCKET);
            HostSlot &victim = slots[(size_t)from * TFE_SLOTS_PER_BUCKET + s];
            std::swap(key, victim.key);
            std::swap(val, victim.val);
            pos[(size_t)(victim.val >> 32)] = (uint32_t)(from * TFE_SLOTS_PER_BUCKET + s);
            avoid = from;
        }
        if (!placed) return false;
    }
    return true;
}

// Grow the per-lookup buffers to hold `entries` (= Q * cols) results.  Not on the hot path:
// only a call with more entries than any earlier one allocates (and synchronises the device).
tfe_status ensure_entries(tfe_ctx *c, int64_t entries)
{
    if (entries <= c->ent_cap) return TFE_OK;
    int64_t cap = std::max<int64_t>(entries, 1024);
    CU(cudaDeviceSynchronize());
    free_dev(c->d_scr_rec);
    free_dev(c->d_miss_q); free_dev(c->d_miss_phrase); free_dev(c->d_miss_tier);
    c->d_scr_rec = nullptr;
    c->d_miss_q = c->d_miss_phrase = nullptr; c->d_miss_tier = nullptr;
    c->ent_cap = 0;
    CU(cudaMalloc(&c->d_scr_rec, cap * 8));
    CU(cudaMemset(c->d_scr_rec, 0, cap * 8));      // tag 0: no call's record
    CU(cudaMalloc(&c->d_miss_q, cap * 4));
    CU(cudaMalloc(&c->d_miss_phrase, cap * 4));
    CU(cudaMalloc(&c->d_miss_tier, cap));
    c->ent_cap = cap;
    return TFE_OK;
}

}  // namespace

extern "C" {

const char *tfe_status_string(tfe_status s)
{
    switch (s) {
    case TFE_OK: return "ok";
    case TFE_ERR_INVALID_ARG: return "invalid argument";
    case TFE_ERR_DUPLICATE_PHRASE: return "duplicate phrase";
    case TFE_ERR_KEY_COLLISION: return "64-bit key collision between two phrases";
    case TFE_ERR_CAPACITY: return "index capacity exceeded";
    case TFE_ERR_SLOT_RANGE: return "GPU-tier slot out of range or used twice";
    case TFE_ERR_UNKNOWN_PHRASE: return "unknown phrase id";
    case TFE_ERR_ALREADY_RESIDENT: return "phrase is already GPU-resident";
    case TFE_ERR_MISS_OVERFLOW: return "miss list larger than the caller's buffers";
    case TFE_ERR_PROBE_LIMIT: return "probe limit reached while building the index";
    case TFE_ERR_CUDA: return "CUDA runtime error";
    case TFE_ERR_INTERNAL: return "bounded device-side wait expired";
    }
    return "unknown status";
}

const char *tfe_last_cuda_error(void) { return g_cuda_error.c_str(); }

uint64_t tfe_phrase_key64(int32_t vocab, const int32_t *tokens, int32_t n, int32_t *is_exact)
{
    if (vocab < 1 || n < 1 || n > 4 || !tokens) return 0;
    const int bits = tfe_token_bits(vocab);
    int32_t tk[4] = {-1, -1, -1, -1};
    for (int j = 0; j < n; ++j) {
        int32_t x = tokens[n - 1 - j];
        if (x < 0 || x >= vocab) return 0;
        tk[j] = x;
    }
    if (is_exact) *is_exact = tfe_order_is_packed(n, bits) ? 1 : 0;
    return tfe_make_key(n, tk, bits);
}

uint64_t tfe_home_bucket(uint64_t key, uint64_t n_buckets)
{
    return n_buckets ? tfe_home_bucket_of(key, n_buckets) : 0;
}

void tfe_destroy(tfe_ctx *c)
{
    if (!c) return;
    int prev = 0;
    (void)cudaGetDevice(&prev);
    (void)cudaSetDevice(c->device);
    (void)cudaDeviceSynchronize();
    if (c->d_arena) {
        free_dev(c->d_arena);
    } else {
        free_dev(c->d_index); free_dev(c->d_phrase_tokens); free_dev(c->d_phrase_pos);
        free_dev(c->d_slot_owner); free_dev(c->d_counters);
    }
    free_dev(c->d_scr_rec);
    free_dev(c->d_miss_q); free_dev(c->d_miss_phrase); free_dev(c->d_miss_tier);
    free_dev(c->d_inst_ids); free_dev(c->d_inst_slots); free_dev(c->d_inst_rows);
    free_dev(c->d_h_tokens); free_dev(c->d_h_hidden); free_dev(c->d_h_out);
    free_dev(c->d_h_phrase); free_dev(c->d_h_slot); free_dev(c->d_h_flag);
    free_dev(c->d_pf_keys); free_dev(c->d_pf_phrase); free_dev(c->d_pf_tier); free_dev(c->d_pf_counter);
    free_dev(c->d_phrase_stamp); free_dev(c->d_slot_stamp); free_dev(c->d_inst_count); free_dev(c->d_inst_flags);
    free_dev(c->d_slot_stats); free_dev(c->d_epoch); free_dev(c->d_vs_fin);
    free_dev(c->d_vs_keys); free_dev(c->d_vs_state); free_dev(c->d_vs_list); free_dev(c->d_vs_slots);
    if (c->hb_in) (void)cudaStreamDestroy(c->hb_in);
    if (c->hb_out) (void)cudaStreamDestroy(c->hb_out);
    if (c->hb_ev_start) (void)cudaEventDestroy(c->hb_ev_start);
    if (c->hb_ev_done) (void)cudaEventDestroy(c->hb_ev_done);
    for (int k = 0; k < tfe_ctx::kPipeMaxChunks; ++k) {
        if (c->hb_ev_in[k]) (void)cudaEventDestroy(c->hb_ev_in[k]);
        if (c->hb_ev_k[k]) (void)cudaEventDestroy(c->hb_ev_k[k]);
    }
    (void)cudaSetDevice(prev);
    delete c;
}

tfe_status tfe_index_build(const tfe_config *cfg, const int32_t *phrase_tokens,
                           const uint8_t *phrase_len, const int32_t *init_slot, void *gpu_rows,
                           void *stream_, tfe_ctx **out)
{
    if (!out) return TFE_ERR_INVALID_ARG;
    *out = nullptr;
    tfe_status st = validate_config(cfg);
    if (st != TFE_OK) return st;
    const int64_t N = cfg->n_phrases, C = cfg->gpu_slots;
    if (N > 0 && (!phrase_tokens || !phrase_len || !init_slot)) return TFE_ERR_INVALID_ARG;
    if (C > 0 && !gpu_rows) return TFE_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(gpu_rows) & 15u) != 0) return TFE_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);

    const int bits = tfe_token_bits(cfg->vocab);
    bool order_ok[5] = {false, false, false, false, false};
    bool any_hashed = false;
    for (int i = 0; i < cfg->n_orders; ++i) {
        order_ok[cfg->orders[i]] = true;
        any_hashed |= !tfe_order_is_packed(cfg->orders[i], bits);
    }

    // ---- host-side checks and key formation
    std::vector<uint64_t> keys((size_t)N);
    std::vector<uint32_t> owner((size_t)C, kNoOwner);
    for (int64_t i = 0; i < N; ++i) {
        const int n = phrase_len[i];
        if (n < 1 || n > 4 || !order_ok[n]) return TFE_ERR_INVALID_ARG;
        int32_t tk[4] = {-1, -1, -1, -1};
        for (int j = 0; j < n; ++j) {
            const int32_t x = phrase_tokens[i * 4 + (n - 1 - j)];
            if (x < 0 || x >= cfg->vocab) return TFE_ERR_INVALID_ARG;
            tk[j] = x;
        }
        keys[(size_t)i] = tfe_make_key(n, tk, bits);
        const int32_t s = init_slot[i];
        if (s >= 0) {
            if (s >= C || owner[(size_t)s] != kNoOwner) return TFE_ERR_SLOT_RANGE;
            owner[(size_t)s] = (uint32_t)i;
        } else if (s != -1 && s != -2) {
            return TFE_ERR_INVALID_ARG;
        }
    }
    {   // equal keys: the same tuple twice, or (hashed orders only) two tuples on one key
        std::vector<std::pair<uint64_t, uint32_t>> sorted((size_t)N);
        for (int64_t i = 0; i < N; ++i) sorted[(size_t)i] = {keys[(size_t)i], (uint32_t)i};
        std::sort(sorted.begin(), sorted.end());
        for (int64_t i = 1; i < N; ++i) {
            if (sorted[(size_t)i].first != sorted[(size_t)i - 1].first) continue;
            const uint32_t a = sorted[(size_t)i].second, b = sorted[(size_t)i - 1].second;
            const bool same = phrase_len[a] == phrase_len[b] &&
                              std::memcmp(phrase_tokens + (size_t)a * 4, phrase_tokens + (size_t)b * 4,
                                          sizeof(int32_t) * phrase_len[a]) == 0;
            return same ? TFE_ERR_DUPLICATE_PHRASE : TFE_ERR_KEY_COLLISION;
        }
    }
    const double want_slots = std::max<double>(1.0, (double)N / (double)cfg->load_factor);
    const uint64_t n_buckets =
        std::max<uint64_t>(1, (uint64_t)((want_slots + TFE_SLOTS_PER_BUCKET - 1) / TFE_SLOTS_PER_BUCKET));
    if (n_buckets * TFE_SLOTS_PER_BUCKET > 0xFFFFFFFFull) return TFE_ERR_CAPACITY;
    if ((uint64_t)N > n_buckets * TFE_SLOTS_PER_BUCKET) return TFE_ERR_CAPACITY;

    // ---- device state
    tfe_ctx *c = new (std::nothrow) tfe_ctx();
    if (!c) return TFE_ERR_INVALID_ARG;
    c->cfg = *cfg;
    c->tok_bits = bits;
    c->any_hashed = any_hashed;
    c->n_buckets = n_buckets;
    c->row_vecs = cfg->d / 8;
    c->gpu_rows = static_cast<uint4 *>(gpu_rows);
    c->h_slot.assign(init_slot, init_slot + N);
    c->h_owner.swap(owner);

    tfe_status rc = TFE_OK;
    auto fail = [&](tfe_status s) {
        tfe_destroy(c);
        return s;
    };
#define CUF(call)                                                  \
    do {                                                           \
        if (cuda_failed((call), #call)) return fail(TFE_ERR_CUDA); \
    } while (0)
    std::vector<HostSlot> slots;
    std::vector<uint32_t> pos;
    if (!cuckoo_build(keys, init_slot, n_buckets, cfg->max_kicks > 0 ? cfg->max_kicks : kDefaultMaxKicks, slots, pos))
        return fail(TFE_ERR_PROBE_LIMIT);
    CUF(cudaGetDevice(&c->device));
    CUF(cudaDeviceGetAttribute(&c->sm_count, cudaDevAttrMultiProcessorCount, c->device));
    const size_t index_bytes = (size_t)n_buckets * TFE_SLOTS_PER_BUCKET * sizeof(ulonglong2);
    CUF(cudaMalloc(&c->d_index, index_bytes));
    CUF(cudaMemcpyAsync(c->d_index, slots.data(), index_bytes, cudaMemcpyHostToDevice, stream));
    CUF(cudaMalloc(&c->d_phrase_pos, std::max<size_t>(4, (size_t)N * 4)));
    if (N > 0) CUF(cudaMemcpyAsync(c->d_phrase_pos, pos.data(), (size_t)N * 4, cudaMemcpyHostToDevice, stream));
    CUF(cudaMalloc(&c->d_slot_owner, std::max<size_t>(4, (size_t)(C + 3) / 4 * 4) * 4));      // whole 16-byte groups
    CUF(cudaMalloc(&c->d_counters, TFE_CTR_WORDS * sizeof(uint32_t)));
    CUF(cudaMemsetAsync(c->d_counters, 0, TFE_CTR_WORDS * sizeof(uint32_t), stream));
    if (C > 0)
        CUF(cudaMemcpyAsync(c->d_slot_owner, c->h_owner.data(), (size_t)C * 4, cudaMemcpyHostToDevice, stream));
    if (any_hashed && N > 0) {
        CUF(cudaMalloc(&c->d_phrase_tokens, (size_t)N * sizeof(int4)));
        CUF(cudaMemcpyAsync(c->d_phrase_tokens, phrase_tokens, (size_t)N * sizeof(int4),
                            cudaMemcpyHostToDevice, stream));
    }
    CUF(lookup_occupancy(c->device, c->occ));
    CUF(cudaStreamSynchronize(stream));
    if (rc != TFE_OK) return fail(rc);
    CUF(cudaMemsetAsync(c->d_counters, 0, TFE_CTR_WORDS * sizeof(uint32_t), stream));
    CUF(cudaStreamSynchronize(stream));
#undef CUF
    *out = c;
    return TFE_OK;
}

tfe_status tfe_index_build_device(const tfe_config *cfg, const int32_t *phrase_tokens,
                                  const uint8_t *phrase_len, const int32_t *init_slot, void *gpu_rows,
                                  void *stream_, tfe_ctx **out)
{
    if (!out) return TFE_ERR_INVALID_ARG;
    *out = nullptr;
    tfe_status st = validate_config(cfg);
    if (st != TFE_OK) return st;
    const int64_t N = cfg->n_phrases, C = cfg->gpu_slots;
    if (N > 0 && (!phrase_tokens || !phrase_len || !init_slot)) return TFE_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(phrase_tokens) & 15u) != 0) return TFE_ERR_INVALID_ARG;
    if (C > 0 && !gpu_rows) return TFE_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(gpu_rows) & 15u) != 0) return TFE_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const int bits = tfe_token_bits(cfg->vocab);
    uint32_t order_mask = 0, hashed_mask = 0;
    for (int i = 0; i < cfg->n_orders; ++i) {
        order_mask |= 1u << cfg->orders[i];
        if (!tfe_order_is_packed(cfg->orders[i], bits)) hashed_mask |= 1u << cfg->orders[i];
    }
    const double want_slots = std::max<double>(1.0, (double)N / (double)cfg->load_factor);
    const uint64_t n_buckets =
        std::max<uint64_t>(1, (uint64_t)((want_slots + TFE_SLOTS_PER_BUCKET - 1) / TFE_SLOTS_PER_BUCKET));
    if (n_buckets * TFE_SLOTS_PER_BUCKET > 0xFFFFFFFFull) return TFE_ERR_CAPACITY;
    if ((uint64_t)N > n_buckets * TFE_SLOTS_PER_BUCKET) return TFE_ERR_CAPACITY;

    tfe_ctx *c = new (std::nothrow) tfe_ctx();
    if (!c) return TFE_ERR_INVALID_ARG;
    c->cfg = *cfg;
    c->tok_bits = bits;
    c->any_hashed = hashed_mask != 0;
    c->n_buckets = n_buckets;
    c->row_vecs = cfg->d / 8;
    c->gpu_rows = static_cast<uint4 *>(gpu_rows);
    uint32_t *d_status = nullptr;
    auto fail = [&](tfe_status s) {
        tfe_destroy(c);
        return s;
    };
#define CUF(call)                                                  \
    do {                                                           \
        if (cuda_failed((call), #call)) return fail(TFE_ERR_CUDA); \
    } while (0)
    CUF(cudaGetDevice(&c->device));
    CUF(cudaDeviceGetAttribute(&c->sm_count, cudaDevAttrMultiProcessorCount, c->device));
    const size_t n_slots = (size_t)n_buckets * TFE_SLOTS_PER_BUCKET;
    const size_t owner_entries = std::max<size_t>(4, (size_t)(C + 3) / 4 * 4);
    {
        // one allocation for everything the build fills (several cost most of a millisecond each at these sizes)
        auto round = [](size_t b) { return (b + 255) & ~(size_t)255; };
        const size_t b_index = round(n_slots * sizeof(ulonglong2)), b_pos = round(std::max<size_t>(4, (size_t)N * 4));
        const size_t b_owner = round(owner_entries * 4), b_ctr = round((TFE_CTR_WORDS + 1) * sizeof(uint32_t));
        const size_t b_tok = c->any_hashed && N > 0 ? round((size_t)N * sizeof(int4)) : 0;
        CUF(cudaMalloc(&c->d_arena, b_index + b_pos + b_owner + b_ctr + b_tok));
        char *at = static_cast<char *>(c->d_arena);
        c->d_index = reinterpret_cast<ulonglong2 *>(at); at += b_index;
        c->d_phrase_pos = reinterpret_cast<uint32_t *>(at); at += b_pos;
        c->d_slot_owner = reinterpret_cast<uint32_t *>(at); at += b_owner;
        c->d_counters = reinterpret_cast<uint32_t *>(at);
        d_status = c->d_counters + TFE_CTR_WORDS; at += b_ctr;
        if (b_tok) c->d_phrase_tokens = reinterpret_cast<int4 *>(at);
    }
    CUF(cudaMemsetAsync(c->d_index, 0, n_slots * sizeof(ulonglong2), stream));
    CUF(cudaMemsetAsync(c->d_slot_owner, 0xFF, owner_entries * 4, stream));
    CUF(cudaMemsetAsync(c->d_counters, 0, TFE_CTR_WORDS * sizeof(uint32_t), stream));
    CUF(cudaMemsetAsync(d_status, 0, sizeof(uint32_t), stream));
    if (c->d_phrase_tokens)
        CUF(cudaMemcpyAsync(c->d_phrase_tokens, phrase_tokens, (size_t)N * sizeof(int4), cudaMemcpyDeviceToDevice, stream));
    TfeBuildParams b{};
    b.phrase_tokens = reinterpret_cast<const int4 *>(phrase_tokens);
    b.phrase_len = phrase_len; b.init_slot = init_slot;
    b.n_phrases = (uint32_t)N; b.gpu_slots = C; b.vocab = cfg->vocab; b.tok_bits = bits;
    b.order_mask = order_mask; b.hashed_mask = hashed_mask;
    b.max_kicks = cfg->max_kicks > 0 ? cfg->max_kicks : kDefaultMaxKicks;
    b.index = c->d_index; b.n_buckets = n_buckets;
    b.slot_owner = c->d_slot_owner; b.phrase_pos = c->d_phrase_pos; b.status = d_status;
    uint32_t status = 0;
    if (N > 0) {
        const unsigned blocks = (unsigned)((N + 255) / 256);
        tfe_build_insert_kernel<<<blocks, 256, 0, stream>>>(b);
        tfe_build_verify_kernel<<<blocks, 256, 0, stream>>>(b);
        CUF(cudaGetLastError());
        CUF(cudaMemcpyAsync(&status, d_status, sizeof status, cudaMemcpyDeviceToHost, stream));
    }
    c->mirror_ready = false;        // the host mirror of the residency state is fetched when tfe_cache_install first needs it
    CUF(lookup_occupancy(c->device, c->occ));
    CUF(cudaStreamSynchronize(stream));
    if (status & TFE_BUILD_BAD_PHRASE) return fail(TFE_ERR_INVALID_ARG);
    if (status & TFE_BUILD_BAD_SLOT) return fail(TFE_ERR_SLOT_RANGE);
    if (status & TFE_BUILD_DUPLICATE) return fail(TFE_ERR_DUPLICATE_PHRASE);
    if (status & TFE_BUILD_COLLISION) return fail(TFE_ERR_KEY_COLLISION);
    if (status & TFE_BUILD_KICKS) return fail(TFE_ERR_PROBE_LIMIT);
    if (status & TFE_BUILD_LOST) return fail(TFE_ERR_INTERNAL);
#undef CUF
    *out = c;
    return TFE_OK;
}

tfe_status tfe_index_geometry(const tfe_ctx *c, int64_t *n_buckets, int64_t *index_bytes,
                              int64_t *metadata_bytes)
{
    if (!c) return TFE_ERR_INVALID_ARG;
    if (n_buckets) *n_buckets = (int64_t)c->n_buckets;
    if (index_bytes) *index_bytes = (int64_t)(c->n_buckets * TFE_SLOTS_PER_BUCKET * sizeof(ulonglong2));
    if (metadata_bytes)
        *metadata_bytes = c->cfg.n_phrases * 4 + c->cfg.gpu_slots * 4 +
                          (c->any_hashed ? c->cfg.n_phrases * (int64_t)sizeof(int4) : 0);
    return TFE_OK;
}


tfe_status tfe_stream_copy(void *dst, const void *src, int64_t bytes, void *stream_)
{
    if (bytes < 0 || (bytes & 15) != 0) return TFE_ERR_INVALID_ARG;
    if (bytes == 0) return TFE_OK;
    if (!dst || !src || ((reinterpret_cast<uintptr_t>(dst) | reinterpret_cast<uintptr_t>(src)) & 15u) != 0)
        return TFE_ERR_INVALID_ARG;
    int dev = 0, sms = 0;
    CU(cudaGetDevice(&dev));
    CU(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    const size_t n = (size_t)bytes / 16;
    const unsigned grid = (unsigned)std::max<size_t>(1, std::min<size_t>((size_t)sms * 16, (n + 255) / 256));
    tfe_stream_copy_kernel<<<grid, 256, 0, static_cast<cudaStream_t>(stream_)>>>(
        static_cast<const uint4 *>(src), static_cast<uint4 *>(dst), n);
    CU(cudaGetLastError());
    return TFE_OK;
}

tfe_status tfe_set_tuning(tfe_ctx *c, int32_t batch_queries)
{
    if (!c || batch_queries < 0 || batch_queries > 8) return TFE_ERR_INVALID_ARG;
    c->qb_override = batch_queries;
    return TFE_OK;
}

tfe_status tfe_launch_geometry(const tfe_ctx *c, int32_t *grid, int32_t *block, int32_t *batch_queries)
{
    if (!c) return TFE_ERR_INVALID_ARG;
    if (grid) *grid = c->last_grid;
    if (block) *block = c->last_block;
    if (batch_queries) *batch_queries = c->last_qb;
    return TFE_OK;
}

namespace {

// Host mirror {phrase -> residency, slot -> owner} of a context built on the device, read back
// from the index; synchronises the stream.
tfe_status fetch_mirror(tfe_ctx *c, cudaStream_t stream)
{
    const int64_t N = c->cfg.n_phrases, C = c->cfg.gpu_slots;
    c->h_slot.resize((size_t)N);
    c->h_owner.resize((size_t)C);
    int32_t *d_res = nullptr;
    if (N > 0) {
        CU(cudaMalloc(&d_res, (size_t)N * 4));
        tfe_gather_residency_kernel<<<(unsigned)((N + 255) / 256), 256, 0, stream>>>(c->d_index, c->d_phrase_pos,
                                                                                  (uint32_t)N, d_res);
        const cudaError_t e1 = cudaMemcpyAsync(c->h_slot.data(), d_res, (size_t)N * 4, cudaMemcpyDeviceToHost, stream);
        const cudaError_t e2 = cudaStreamSynchronize(stream);
        (void)cudaFree(d_res);
        if (cuda_failed(e1, "copy of the residency mirror") || cuda_failed(e2, "cudaStreamSynchronize")) return TFE_ERR_CUDA;
    }
    if (C > 0) {
        CU(cudaMemcpyAsync(c->h_owner.data(), c->d_slot_owner, (size_t)C * 4, cudaMemcpyDeviceToHost, stream));
        CU(cudaStreamSynchronize(stream));
    }
    c->mirror_ready = !c->device_installs;
    return TFE_OK;
}

}  // namespace

tfe_status tfe_cache_install(tfe_ctx *c, int32_t n, const uint32_t *phrase_ids, const void *src_rows,
                             const int32_t *dst_slots, void *stream_)
{
    if (!c || n < 0) return TFE_ERR_INVALID_ARG;
    if (n == 0) return TFE_OK;
    if (!phrase_ids || !src_rows || !dst_slots) return TFE_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(src_rows) & 15u) != 0) return TFE_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const int64_t N = c->cfg.n_phrases, C = c->cfg.gpu_slots;
    if (!c->mirror_ready) {
        const tfe_status ms = fetch_mirror(c, stream);
        if (ms != TFE_OK) return ms;
    }
    cudaPointerAttributes attr{};
    bool src_on_device = false;
    if (cudaPointerGetAttributes(&attr, src_rows) == cudaSuccess)
        src_on_device = attr.type == cudaMemoryTypeDevice || attr.type == cudaMemoryTypeManaged;
    else
        (void)cudaGetLastError();

    if (n > c->inst_cap) {      // staging grows outside the steady state
        CU(cudaDeviceSynchronize());
        free_dev(c->d_inst_ids); free_dev(c->d_inst_slots); free_dev(c->d_inst_rows);
        c->d_inst_ids = nullptr; c->d_inst_slots = nullptr; c->d_inst_rows = nullptr;
        c->inst_cap = 0;
        CU(cudaMalloc(&c->d_inst_ids, (size_t)n * 4));
        CU(cudaMalloc(&c->d_inst_slots, (size_t)n * 4));
        CU(cudaMalloc(&c->d_inst_rows, (size_t)n * c->row_vecs * sizeof(uint4)));
        c->inst_cap = n;
    }
    // The rows start travelling before the arguments are checked: the copy into the staging area
    // changes nothing a caller can see, and the checks below (a few tens of microseconds for
    // thousands of rows) run while it is under way.
    const uint4 *src = static_cast<const uint4 *>(src_rows);
    if (!src_on_device) {
        CU(cudaMemcpyAsync(c->d_inst_rows, src_rows, (size_t)n * c->row_vecs * sizeof(uint4),
                           cudaMemcpyHostToDevice, stream));
        src = c->d_inst_rows;
    }
    for (int32_t k = 0; k < n; ++k) {
        if ((int64_t)phrase_ids[k] >= N) return TFE_ERR_UNKNOWN_PHRASE;
        if (c->h_slot[phrase_ids[k]] >= 0) return TFE_ERR_ALREADY_RESIDENT;
        if (dst_slots[k] < 0 || dst_slots[k] >= C) return TFE_ERR_SLOT_RANGE;
    }
    {
        std::vector<uint32_t> a(phrase_ids, phrase_ids + n);
        std::vector<int32_t> b(dst_slots, dst_slots + n);
        std::sort(a.begin(), a.end());
        std::sort(b.begin(), b.end());
        if (std::adjacent_find(a.begin(), a.end()) != a.end()) return TFE_ERR_INVALID_ARG;
        if (std::adjacent_find(b.begin(), b.end()) != b.end()) return TFE_ERR_INVALID_ARG;
    }
    CU(cudaMemcpyAsync(c->d_inst_ids, phrase_ids, (size_t)n * 4, cudaMemcpyHostToDevice, stream));
    CU(cudaMemcpyAsync(c->d_inst_slots, dst_slots, (size_t)n * 4, cudaMemcpyHostToDevice, stream));
    const unsigned blocks = (unsigned)((n + TFE_WARPS_PER_BLOCK - 1) / TFE_WARPS_PER_BLOCK);
    tfe_install_kernel<<<blocks, TFE_BLOCK_THREADS, 0, stream>>>(c->d_index, c->d_phrase_pos, c->d_slot_owner,
                                                                 c->gpu_rows, c->row_vecs, n, c->d_inst_ids,
                                                                 src, c->d_inst_slots, c->d_slot_stats, c->d_epoch);
    CU(cudaGetLastError());
    for (int32_t k = 0; k < n; ++k) {       // mirror, same order as the oracle's state machine
        const uint32_t prev = c->h_owner[(size_t)dst_slots[k]];
        if (prev != kNoOwner) c->h_slot[prev] = -1;
        c->h_slot[phrase_ids[k]] = dst_slots[k];
        c->h_owner[(size_t)dst_slots[k]] = phrase_ids[k];
    }
    return TFE_OK;
}

tfe_status tfe_cache_install_device(tfe_ctx *c, int32_t n, const uint32_t *phrase_ids, const void *src_rows,
                                    const int32_t *dst_slots, uint8_t *applied, uint32_t *applied_count,
                                    void *stream_)
{
    if (!c || n < 0 || n > TFE_INSTALL_DEVICE_MAX) return TFE_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (n == 0) {
        if (applied_count) CU(cudaMemsetAsync(applied_count, 0, sizeof(uint32_t), stream));
        return TFE_OK;
    }
    if (!phrase_ids || !src_rows || !dst_slots) return TFE_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(src_rows) & 15u) != 0) return TFE_ERR_INVALID_ARG;
    const int64_t N = c->cfg.n_phrases, C = c->cfg.gpu_slots;
    if (!c->d_phrase_stamp) {       // first use: the stamp arrays (4 bytes per phrase and per slot)
        CU(cudaDeviceSynchronize());
        CU(cudaMalloc(&c->d_phrase_stamp, std::max<size_t>(4, (size_t)N * 4)));
        CU(cudaMalloc(&c->d_slot_stamp, std::max<size_t>(4, (size_t)C * 4)));
        CU(cudaMalloc(&c->d_inst_count, sizeof(uint32_t)));
        CU(cudaMalloc(&c->d_inst_flags, TFE_INSTALL_DEVICE_MAX));
        // zero once; every call leaves them zeroed again
        CU(cudaMemsetAsync(c->d_phrase_stamp, 0, std::max<size_t>(4, (size_t)N * 4), stream));
        CU(cudaMemsetAsync(c->d_slot_stamp, 0, std::max<size_t>(4, (size_t)C * 4), stream));
    }
    TfeInstallDeviceParams p{};
    p.index = c->d_index; p.phrase_pos = c->d_phrase_pos; p.slot_owner = c->d_slot_owner;
    p.rows = c->gpu_rows; p.row_vecs = c->row_vecs; p.n = n;
    p.n_phrases = (uint32_t)N; p.gpu_slots = C;
    p.ids = phrase_ids; p.src = static_cast<const uint4 *>(src_rows); p.dst_slots = dst_slots;
    p.phrase_stamp = c->d_phrase_stamp; p.slot_stamp = c->d_slot_stamp;
    p.applied = applied; p.count = applied_count ? applied_count : c->d_inst_count;
    p.slot_stats = c->d_slot_stats; p.epoch = c->d_epoch;
    p.flags = c->d_inst_flags;
    CU(launch_overlapped(tfe_install_claim_kernel, dim3(1), dim3(TFE_INSTALL_CLAIM_THREADS), stream, p));
    CU(launch_overlapped(tfe_install_device_kernel, dim3((unsigned)((n + TFE_WARPS_PER_BLOCK - 1) / TFE_WARPS_PER_BLOCK)),
                         dim3(TFE_BLOCK_THREADS), stream, p));
    c->mirror_ready = false;        // the host copy of the residency state is stale now; fetched again when needed
    c->device_installs = true;
    return TFE_OK;
}

// Bytes of hidden state per piece of the host-buffer variant's copy / compute pipeline: the
// largest piece, and the smallest (the last ones).
#ifndef TFE_HOST_CHUNK_BYTES
#define TFE_HOST_CHUNK_BYTES ((size_t)8 << 20)
#endif
#ifndef TFE_HOST_TAIL_BYTES
#define TFE_HOST_TAIL_BYTES ((size_t)1 << 20)       // the last two pieces; earlier ones double up to the above
#endif

namespace {

// Variant of the lookup kernel a call runs: the LONGEST / CONST kernels where they apply.
int lookup_variant(const tfe_ctx *c, const tfe_inject_params *prm, int64_t Q)
{
    const bool all = prm->policy == TFE_POLICY_ALL, cos = prm->gate == TFE_GATE_COSINE;
    uint32_t lam_bits;
    std::memcpy(&lam_bits, &prm->lambda, sizeof lam_bits);
    const bool lam_is_bf16 = (lam_bits & 0xFFFFu) == 0 && (lam_bits & 0x7F800000u) != 0x7F800000u;
    const int ht = c->cfg.hidden_dtype;
    // (a decode-sized call is a little quicker in the general kernel: 5.1 against 5.4 us at 64 positions)
    if (!all && cos && c->cfg.d / (ht == 0 ? 8 : 4) <= kCosSteps && Q >= kCosMinQueries) return kVarLongestCos + ht;
    return (all || cos) ? ht * 4 + (all ? 2 : 0) + (cos ? 1 : 0)
                        : (ht == 1 ? kVarLongestF32 : (lam_is_bf16 ? kVarLongestPacked : kVarLongest));
}

tfe_status lookup_inject_range(tfe_ctx *c, const int32_t *tokens, int32_t B, int32_t T, int32_t q_start,
                               const void *h, void *out, const tfe_inject_params *prm,
                               uint32_t *sel_phrase, int32_t *sel_slot, uint8_t *flags, cudaStream_t stream,
                               int64_t q_lo, int64_t q_hi, bool finalize);

// Piece boundaries of the host-buffer pipeline over Q rows: cut[0] = 0 < ... < cut[n] = Q, n returned.
// The first piece's copy-in and the last piece's kernel and copy-back are the exposed parts, in
// between both copy engines stay busy; so pieces are small at both ends (tail, tail, 2 tail,
// 4 tail, ...) and large (few stream hand-overs) in the middle.
int plan_pieces(int64_t Q, int64_t row_bytes, int64_t *cut)
{
    const int max_n = tfe_ctx::kPipeMaxChunks;
    const int64_t tail = std::max<int64_t>(64, (int64_t)TFE_HOST_TAIL_BYTES / row_bytes / 64 * 64);
    int64_t big = std::max<int64_t>(tail, (int64_t)TFE_HOST_CHUNK_BYTES / row_bytes / 64 * 64);
    for (;; big *= 2) {
        int64_t head[max_n], back[max_n];
        int nh = 0, nb = 0;
        int64_t left = Q, next = tail;
        while (left > 0 && nh + nb < max_n) {
            const int64_t a = std::min(left, next);
            head[nh++] = a; left -= a;
            const int64_t b = std::min(left, next);
            if (b > 0 && nh + nb < max_n) { back[nb++] = b; left -= b; }
            if (nh >= 2) next = std::min(big, next * 2);
        }
        if (left > 0) continue;         // too many pieces: larger middle pieces
        for (int k = 0; k < nh; ++k) cut[k + 1] = cut[k] + head[k];
        for (int k = 0; k < nb; ++k) cut[nh + k + 1] = cut[nh + k] + back[nb - 1 - k];
        return nh + nb;
    }
}


}  // namespace

tfe_status tfe_lookup_inject(tfe_ctx *c, const int32_t *tokens, int32_t B, int32_t T, int32_t q_start,
                             const void *h, void *out, const tfe_inject_params *prm,
                             uint32_t *sel_phrase, int32_t *sel_slot, uint8_t *flags, void *stream_)
{
    if (!c || !prm || B < 0 || T < 0 || q_start < 0 || q_start > T) return TFE_ERR_INVALID_ARG;
    if (prm->policy != TFE_POLICY_LONGEST && prm->policy != TFE_POLICY_ALL) return TFE_ERR_INVALID_ARG;
    if (prm->gate != TFE_GATE_CONST && prm->gate != TFE_GATE_COSINE) return TFE_ERR_INVALID_ARG;
    const int64_t Tq = T - q_start, Q = (int64_t)B * Tq;
    const int cols = prm->policy == TFE_POLICY_ALL ? c->cfg.n_orders : 1;
    if (Q * cols > 0x7FFFFFFFll) return TFE_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (Q == 0) {      // nothing to launch; the miss count of "this lookup" is zero
        CU(cudaMemsetAsync(c->d_counters + TFE_CTR_TOTAL, 0, sizeof(uint32_t), stream));
        c->last_entries = 0;
        c->last_grid = 0;
        return TFE_OK;
    }
    if (!tokens || !h || !out) return TFE_ERR_INVALID_ARG;
    if (((reinterpret_cast<uintptr_t>(h) | reinterpret_cast<uintptr_t>(out)) & 15u) != 0)
        return TFE_ERR_INVALID_ARG;
    tfe_status st = ensure_entries(c, Q * cols);
    if (st != TFE_OK) return st;
    return lookup_inject_range(c, tokens, B, T, q_start, h, out, prm, sel_phrase, sel_slot, flags, stream, 0, Q, true);
}

namespace {

// One launch over queries [q_lo, q_hi) of a call of Q queries.  A call issued in several launches
// (LONGEST / CONST kernels only) passes finalize on the last one, which builds the miss list of
// the whole call; the launches must run in order on one stream.
tfe_status lookup_inject_range(tfe_ctx *c, const int32_t *tokens, int32_t B, int32_t T, int32_t q_start,
                               const void *h, void *out, const tfe_inject_params *prm,
                               uint32_t *sel_phrase, int32_t *sel_slot, uint8_t *flags, cudaStream_t stream,
                               int64_t q_lo, int64_t q_hi, bool finalize)
{
    const int64_t Tq = T - q_start, Q = (int64_t)B * Tq;
    const int cols = prm->policy == TFE_POLICY_ALL ? c->cfg.n_orders : 1;
    uint32_t lam_bits;
    std::memcpy(&lam_bits, &prm->lambda, sizeof lam_bits);
    const bool ranged = q_lo != 0 || q_hi != Q || !finalize;
    int variant = lookup_variant(c, prm, Q);
    if (ranged && !is_longest_const(variant)) return TFE_ERR_INTERNAL;
    if (ranged) variant += kVarRanged;
    if (is_longest_const(variant) && c->cfg.d / (c->cfg.hidden_dtype == 0 ? 8 : 4) >= kWideSteps) variant += kVarWide;
    const int64_t Qr = q_hi - q_lo;
    int64_t qb, grid;
    lookup_geometry(c, variant, Qr, &qb, &grid);
    TfeLookupParams p{};
    p.tokens = tokens; p.B = B; p.T = T; p.q_start = q_start; p.Tq = (int32_t)Tq; p.Q = (uint32_t)Q;
    p.div_tq = make_fastdiv((uint32_t)Tq); p.qb = (uint32_t)qb;
    p.q_lo = (uint32_t)q_lo; p.q_hi = (uint32_t)q_hi; p.finalize = finalize ? 1u : 0u;
    p.index = c->d_index; p.n_buckets = c->n_buckets;
    p.phrase_tokens = c->d_phrase_tokens; p.rows = c->gpu_rows; p.d = c->cfg.d;
    p.h = h; p.out = out;
    p.n_orders = c->cfg.n_orders;
    for (int i = 0; i < 4; ++i) p.orders[i] = i < c->cfg.n_orders ? c->cfg.orders[i] : 0;
    p.tok_bits = c->tok_bits; p.vocab = c->cfg.vocab; p.lambda = prm->lambda;
    p.lambda_bf16x2 = (lam_bits >> 16) | (lam_bits & 0xFFFF0000u);
    p.sel_phrase = sel_phrase; p.sel_slot = sel_slot; p.flags = flags;
    p.scr_rec = c->d_scr_rec;
    p.miss_q = c->d_miss_q; p.miss_phrase = c->d_miss_phrase; p.miss_tier = c->d_miss_tier;
    p.counters = c->d_counters;
    p.slot_stats = c->d_slot_stats; p.epoch = c->d_epoch;

    // Programmatic stream serialisation: the launch may be set up while the kernel before it on the
    // stream drains; the kernel itself waits for that kernel's completion before its first global access.
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)grid); cfg.blockDim = dim3(TFE_BLOCK_THREADS); cfg.dynamicSmemBytes = 0; cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    CU(cudaLaunchKernelEx(&cfg, pick_kernel(variant), p));
    CU(cudaGetLastError());
    c->last_entries = Q * cols;
    c->last_grid = (int)grid;
    c->last_block = TFE_BLOCK_THREADS;
    c->last_qb = (int)qb;
    return TFE_OK;
}

}  // namespace

tfe_status tfe_lookup_inject_host(tfe_ctx *c, const int32_t *tokens, int32_t B, int32_t T, int32_t q_start,
                                  const void *h, void *out, const tfe_inject_params *prm,
                                  uint32_t *sel_phrase, int32_t *sel_slot, uint8_t *flags, void *stream_)
{
    if (!c || !prm || B < 0 || T < 0 || q_start < 0 || q_start > T) return TFE_ERR_INVALID_ARG;
    if (prm->policy != TFE_POLICY_LONGEST && prm->policy != TFE_POLICY_ALL) return TFE_ERR_INVALID_ARG;
    if (prm->gate != TFE_GATE_CONST && prm->gate != TFE_GATE_COSINE) return TFE_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const int64_t n_tok = (int64_t)B * T, Q = (int64_t)B * (T - q_start);
    const int cols = prm->policy == TFE_POLICY_ALL ? c->cfg.n_orders : 1;
    const int64_t ent = Q * cols;
    if (Q == 0) return tfe_lookup_inject(c, nullptr, B, T, q_start, nullptr, nullptr, prm, nullptr, nullptr, nullptr, stream_);
    if (!tokens || !h || !out) return TFE_ERR_INVALID_ARG;
    const size_t hid_bytes = (size_t)Q * c->cfg.d * (c->cfg.hidden_dtype == 0 ? 2 : 4);
    if (n_tok > c->hb_tok_cap || Q > c->hb_q_cap || ent > c->hb_ent_cap) {
        // every dimension keeps the larger of what it had and what this call needs, so calls of alternating
        // shapes settle after one regrow each
        const int64_t tok_cap = std::max(n_tok, c->hb_tok_cap), q_cap = std::max(Q, c->hb_q_cap);
        const int64_t e_cap = std::max<int64_t>(std::max(ent, c->hb_ent_cap), q_cap * c->cfg.n_orders);
        CU(cudaDeviceSynchronize());
        free_dev(c->d_h_tokens); free_dev(c->d_h_hidden); free_dev(c->d_h_out);
        free_dev(c->d_h_phrase); free_dev(c->d_h_slot); free_dev(c->d_h_flag);
        c->d_h_tokens = nullptr; c->d_h_hidden = c->d_h_out = nullptr;
        c->d_h_phrase = nullptr; c->d_h_slot = nullptr; c->d_h_flag = nullptr;
        c->hb_tok_cap = c->hb_q_cap = c->hb_ent_cap = 0;
        const size_t row_bytes = (size_t)c->cfg.d * (c->cfg.hidden_dtype == 0 ? 2 : 4);
        CU(cudaMalloc(&c->d_h_tokens, (size_t)tok_cap * 4));
        CU(cudaMalloc(&c->d_h_hidden, (size_t)q_cap * row_bytes));
        CU(cudaMalloc(&c->d_h_out, (size_t)q_cap * row_bytes));
        CU(cudaMalloc(&c->d_h_phrase, (size_t)e_cap * 4));
        CU(cudaMalloc(&c->d_h_slot, (size_t)e_cap * 4));
        CU(cudaMalloc(&c->d_h_flag, (size_t)e_cap));
        c->hb_tok_cap = tok_cap; c->hb_q_cap = q_cap; c->hb_ent_cap = e_cap;
    }
    const size_t row_bytes = (size_t)c->cfg.d * (c->cfg.hidden_dtype == 0 ? 2 : 4);
    const int variant = lookup_variant(c, prm, Q);
    // The LONGEST / CONST kernels can run a call in pieces, so the hidden states go through a
    // three-stage pipeline: piece k's kernel runs while piece k+1 comes in and piece k-1 goes
    // back.  Other variants take one launch between the copies.
    int64_t cut[tfe_ctx::kPipeMaxChunks + 1];
    int n_chunks = 1;
    cut[0] = 0; cut[1] = Q;
    if (is_longest_const(variant) && hid_bytes >= 2 * (size_t)TFE_HOST_CHUNK_BYTES)
        n_chunks = plan_pieces(Q, (int64_t)row_bytes, cut);
    if (n_chunks == 1) {
        CU(cudaMemcpyAsync(c->d_h_tokens, tokens, (size_t)n_tok * 4, cudaMemcpyHostToDevice, stream));
        CU(cudaMemcpyAsync(c->d_h_hidden, h, hid_bytes, cudaMemcpyHostToDevice, stream));
        tfe_status st = tfe_lookup_inject(c, c->d_h_tokens, B, T, q_start, c->d_h_hidden, c->d_h_out, prm,
                                          sel_phrase ? c->d_h_phrase : nullptr, sel_slot ? c->d_h_slot : nullptr,
                                          flags ? c->d_h_flag : nullptr, stream_);
        if (st != TFE_OK) return st;
        CU(cudaMemcpyAsync(out, c->d_h_out, hid_bytes, cudaMemcpyDeviceToHost, stream));
        if (sel_phrase) CU(cudaMemcpyAsync(sel_phrase, c->d_h_phrase, (size_t)ent * 4, cudaMemcpyDeviceToHost, stream));
        if (sel_slot) CU(cudaMemcpyAsync(sel_slot, c->d_h_slot, (size_t)ent * 4, cudaMemcpyDeviceToHost, stream));
        if (flags) CU(cudaMemcpyAsync(flags, c->d_h_flag, (size_t)ent, cudaMemcpyDeviceToHost, stream));
        return TFE_OK;
    }
    if (!c->hb_in) {
        CU(cudaStreamCreateWithFlags(&c->hb_in, cudaStreamNonBlocking));
        CU(cudaStreamCreateWithFlags(&c->hb_out, cudaStreamNonBlocking));
        CU(cudaEventCreateWithFlags(&c->hb_ev_start, cudaEventDisableTiming));
        CU(cudaEventCreateWithFlags(&c->hb_ev_done, cudaEventDisableTiming));
        for (int k = 0; k < tfe_ctx::kPipeMaxChunks; ++k) {
            CU(cudaEventCreateWithFlags(&c->hb_ev_in[k], cudaEventDisableTiming));
            CU(cudaEventCreateWithFlags(&c->hb_ev_k[k], cudaEventDisableTiming));
        }
    }
    tfe_status st = ensure_entries(c, ent);
    if (st != TFE_OK) return st;
    // everything the caller queued on its stream comes first (the staging buffers may be in use)
    CU(cudaEventRecord(c->hb_ev_start, stream));
    CU(cudaStreamWaitEvent(c->hb_in, c->hb_ev_start, 0));
    CU(cudaStreamWaitEvent(c->hb_out, c->hb_ev_start, 0));
    CU(cudaMemcpyAsync(c->d_h_tokens, tokens, (size_t)n_tok * 4, cudaMemcpyHostToDevice, c->hb_in));
    for (int k = 0; k < n_chunks; ++k) {
        const int64_t q_lo = cut[k], q_hi = cut[k + 1], nq = q_hi - q_lo;
        const size_t off = (size_t)q_lo * row_bytes, len = (size_t)nq * row_bytes;
        CU(cudaMemcpyAsync(static_cast<char *>(c->d_h_hidden) + off, static_cast<const char *>(h) + off, len,
                           cudaMemcpyHostToDevice, c->hb_in));
        CU(cudaEventRecord(c->hb_ev_in[k], c->hb_in));
        CU(cudaStreamWaitEvent(stream, c->hb_ev_in[k], 0));
        st = lookup_inject_range(c, c->d_h_tokens, B, T, q_start, c->d_h_hidden, c->d_h_out, prm,
                                 sel_phrase ? c->d_h_phrase : nullptr, sel_slot ? c->d_h_slot : nullptr,
                                 flags ? c->d_h_flag : nullptr, stream, q_lo, q_hi, q_hi == Q);
        if (st != TFE_OK) return st;
        CU(cudaEventRecord(c->hb_ev_k[k], stream));
        CU(cudaStreamWaitEvent(c->hb_out, c->hb_ev_k[k], 0));
        CU(cudaMemcpyAsync(static_cast<char *>(out) + off, static_cast<const char *>(c->d_h_out) + off, len,
                           cudaMemcpyDeviceToHost, c->hb_out));
        if (sel_phrase) CU(cudaMemcpyAsync(sel_phrase + q_lo, c->d_h_phrase + q_lo, (size_t)nq * 4, cudaMemcpyDeviceToHost, c->hb_out));
        if (sel_slot) CU(cudaMemcpyAsync(sel_slot + q_lo, c->d_h_slot + q_lo, (size_t)nq * 4, cudaMemcpyDeviceToHost, c->hb_out));
        if (flags) CU(cudaMemcpyAsync(flags + q_lo, c->d_h_flag + q_lo, (size_t)nq, cudaMemcpyDeviceToHost, c->hb_out));
    }
    // the caller's stream resumes once the last piece is back in host memory
    CU(cudaEventRecord(c->hb_ev_done, c->hb_out));
    CU(cudaStreamWaitEvent(stream, c->hb_ev_done, 0));
    c->last_entries = ent;
    return TFE_OK;
}

tfe_status tfe_miss_list(tfe_ctx *c, uint32_t *q_idx, uint32_t *phrase_id, uint8_t *tier, int64_t cap,
                         int64_t *count, void *stream_)
{
    if (!c || !count || cap < 0) return TFE_ERR_INVALID_ARG;
    if (cap > 0 && (!q_idx || !phrase_id || !tier)) return TFE_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    *count = 0;
    if (c->last_entries <= 0) {
        CU(cudaStreamSynchronize(stream));
        return c->last_entries < 0 ? TFE_ERR_INVALID_ARG : TFE_OK;
    }
    uint32_t words[TFE_CTR_WORDS] = {0};
    CU(cudaMemcpyAsync(words, c->d_counters, sizeof words, cudaMemcpyDeviceToHost, stream));
    CU(cudaStreamSynchronize(stream));
    if (words[TFE_CTR_STATUS] & TFE_DEV_RECORD_TIMEOUT) return TFE_ERR_INTERNAL;      // the closing block gave up waiting
    const int64_t n = words[TFE_CTR_TOTAL];
    *count = n;
    const int64_t take = std::min(n, cap);
    if (take > 0) {
        CU(cudaMemcpyAsync(q_idx, c->d_miss_q, (size_t)take * 4, cudaMemcpyDeviceToHost, stream));
        CU(cudaMemcpyAsync(phrase_id, c->d_miss_phrase, (size_t)take * 4, cudaMemcpyDeviceToHost, stream));
        CU(cudaMemcpyAsync(tier, c->d_miss_tier, (size_t)take, cudaMemcpyDeviceToHost, stream));
        CU(cudaStreamSynchronize(stream));
    }
    return n > cap ? TFE_ERR_MISS_OVERFLOW : TFE_OK;
}

tfe_status tfe_miss_list_device(tfe_ctx *c, const uint32_t **q_idx, const uint32_t **phrase_id,
                                const uint8_t **tier, const uint32_t **count)
{
    if (!c || c->last_entries < 0) return TFE_ERR_INVALID_ARG;
    if (q_idx) *q_idx = c->d_miss_q;
    if (phrase_id) *phrase_id = c->d_miss_phrase;
    if (tier) *tier = c->d_miss_tier;
    if (count) *count = c->d_counters + TFE_CTR_TOTAL;
    return TFE_OK;
}

tfe_status tfe_cache_policy_enable(tfe_ctx *c, void *stream_)
{
    if (!c) return TFE_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const size_t C = ((size_t)std::max<int64_t>(1, c->cfg.gpu_slots) + 3) / 4 * 4;     // whole 16-byte groups
    if (!c->d_slot_stats) {
        CU(cudaDeviceSynchronize());        // no lookup in flight while the kernels' arguments change
        uint2 *stats = nullptr;
        CU(cudaMalloc(&stats, C * sizeof(uint2)));
        CU(cudaMalloc(&c->d_epoch, sizeof(uint32_t)));
        CU(cudaMalloc(&c->d_vs_state, sizeof(TfeVictimState)));
        CU(cudaMalloc(&c->d_vs_list, (size_t)TFE_VS_LIST_CAP * sizeof(unsigned long long)));
        CU(cudaMalloc(&c->d_vs_fin, (size_t)TFE_VS_FINAL_CAP * sizeof(unsigned long long)));
        CU(cudaFuncSetAttribute(tfe_victim_select_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, TFE_VS_DYN_SMEM));
        CU(cudaFuncSetAttribute(tfe_victim_select_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, TFE_VS_DYN_SMEM));
        int per_sm = 0, per_sm_plain = 0;
        CU(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, tfe_victim_select_kernel<true>, TFE_VS_THREADS, TFE_VS_DYN_SMEM));
        CU(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm_plain, tfe_victim_select_kernel<false>, TFE_VS_THREADS, TFE_VS_DYN_SMEM));
        if (per_sm < 1 || per_sm_plain < 1) return TFE_ERR_INTERNAL;
        c->vs_grid_max = c->sm_count;       // one block per SM: the blocks of the launch wait for one another
        CU(cudaMalloc(&c->d_vs_slots, TFE_VICTIMS_MAX * sizeof(int32_t)));
        CU(cudaMalloc(&c->d_vs_keys, TFE_VICTIMS_MAX * sizeof(uint32_t)));
        c->d_slot_stats = stats;
    }
    tfe_policy_reset_kernel<<<(unsigned)std::min<size_t>(4096, (C + 255) / 256), 256, 0, stream>>>(c->d_slot_stats, c->d_slot_owner,
                                                                                                    (uint32_t)C);
    CU(cudaGetLastError());
    CU(cudaMemsetAsync(c->d_epoch, 0, sizeof(uint32_t), stream));
    CU(cudaMemsetAsync(c->d_vs_state, 0, sizeof(TfeVictimState), stream));
    return TFE_OK;
}

tfe_status tfe_cache_select_victims(tfe_ctx *c, int32_t n, int32_t half_life, int32_t *slots, uint32_t *keys,
                                    int32_t *count, void *stream_)
{
    if (!c || n < 0 || n > TFE_VICTIMS_MAX || !count || half_life > TFE_HALF_LIFE_MAX) return TFE_ERR_INVALID_ARG;
    if (!c->d_slot_stats) return TFE_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const int64_t C = c->cfg.gpu_slots;
    const int32_t take = (int32_t)std::min<int64_t>(n, C);
    *count = take;
    if (take == 0) return TFE_OK;
    TfeVictimParams p{};
    p.slot_stats = c->d_slot_stats; p.epoch = c->d_epoch;
    p.div_half_life = make_fastdiv(half_life > 0 ? (uint32_t)half_life : 1u);
    p.age_cap = half_life > 0 ? 32u * (uint32_t)half_life : 0u;
    p.C = (uint32_t)C; p.take = (uint32_t)take;
    p.list_cap = (uint32_t)(c->vs_list_cap > 0 ? c->vs_list_cap : TFE_VS_LIST_CAP);
    p.final_cap = (uint32_t)std::max<int32_t>(take + 1, c->vs_final_cap > 0 ? c->vs_final_cap : TFE_VS_FINAL_DEFAULT);
    p.range_cap = c->vs_final_cap > 0 ? (uint32_t)std::max(1, std::min(c->vs_final_cap / 2, TFE_VS_FINAL_CAP - TFE_VICTIMS_MAX))
                                      : (uint32_t)TFE_VS_RANGE_DEFAULT;
    if (C > (int64_t)std::min(p.list_cap, p.final_cap)) {     // else: the whole table goes to the final step
        // a threshold from S sampled slots: the take-th smallest number has rank ~ Poisson(mu) among them,
        // mu = take * S / C; the rank used is six standard deviations and a margin above that
        // (S by default: about three samples expected below the take-th smallest -- more only make the merge longer)
        int64_t S = TFE_VS_SAMPLES;
        while (S > 64 && (double)take * (double)(S / 2) / (double)C >= 3.0) S /= 2;
        if (c->vs_samples > 0) S = c->vs_samples;
        S = std::min<int64_t>(C, S);
        const double mu = (double)take * (double)S / (double)C;
        p.n_samples = (uint32_t)S;
        p.sample_stretch = (uint32_t)(C / S); p.sample_longer = (uint32_t)(C % S);
        p.sample_rank = (uint32_t)std::min<double>((double)S, std::ceil(mu + 6.0 * std::sqrt(mu) + 6.0));
    }
    p.list = c->d_vs_list; p.fin = c->d_vs_fin; p.st = c->d_vs_state;
    p.out_slots = c->d_vs_slots; p.out_keys = c->d_vs_keys;
    {
        const int64_t n_quads = (C + 3) / 4;
        cudaLaunchConfig_t cfg{};
        // a small table keeps at least 32 blocks: the final step's cost is shared by the blocks, whatever the table's size
        cfg.gridDim = dim3((unsigned)std::max<int64_t>(std::min(32, c->vs_grid_max), std::min<int64_t>(c->vs_grid_max, (n_quads + TFE_VS_THREADS - 1) / TFE_VS_THREADS)));
        if (take > 512) cfg.gridDim = dim3((unsigned)c->vs_grid_max);
        cfg.blockDim = dim3(TFE_VS_THREADS); cfg.dynamicSmemBytes = TFE_VS_DYN_SMEM; cfg.stream = stream;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeCooperative;      // the blocks wait for one another: resident together
        attr[0].val.cooperative = 1;
        cfg.attrs = attr; cfg.numAttrs = 1;
        CU(cudaLaunchKernelEx(&cfg, half_life > 0 ? tfe_victim_select_kernel<true> : tfe_victim_select_kernel<false>, p));
    }
    CU(cudaGetLastError());
    if (!slots) return TFE_OK;      // results stay on the device (tfe_cache_select_victims_device); no synchronisation
    CU(cudaMemcpyAsync(slots, c->d_vs_slots, (size_t)take * 4, cudaMemcpyDeviceToHost, stream));
    if (keys) CU(cudaMemcpyAsync(keys, c->d_vs_keys, (size_t)take * 4, cudaMemcpyDeviceToHost, stream));
    uint32_t dev_status = 0;
    CU(cudaMemcpyAsync(&dev_status, &c->d_vs_state->status, sizeof(uint32_t), cudaMemcpyDeviceToHost, stream));
    CU(cudaStreamSynchronize(stream));
    if (dev_status) {                       // the launch gave up and left its work space as it was
        CU(cudaMemsetAsync(c->d_vs_state, 0, sizeof(TfeVictimState), stream));
        CU(cudaStreamSynchronize(stream));
        return TFE_ERR_INTERNAL;
    }
    return TFE_OK;
}

tfe_status tfe_cache_select_tuning(tfe_ctx *c, int32_t list_cap, int32_t final_cap, int32_t n_samples)
{
    if (!c || list_cap > TFE_VS_LIST_CAP || final_cap > TFE_VS_FINAL_CAP || n_samples > TFE_VS_SAMPLES) return TFE_ERR_INVALID_ARG;
    c->vs_list_cap = std::max(0, list_cap);
    c->vs_final_cap = std::max(0, final_cap);
    c->vs_samples = std::max(0, n_samples);
    return TFE_OK;
}

tfe_status tfe_cache_select_victims_device(tfe_ctx *c, const int32_t **slots, const uint32_t **keys)
{
    if (!c || !c->d_slot_stats) return TFE_ERR_INVALID_ARG;
    if (slots) *slots = c->d_vs_slots;
    if (keys) *keys = c->d_vs_keys;
    return TFE_OK;
}

tfe_status tfe_cache_stats(tfe_ctx *c, uint32_t *freq_last, uint32_t *epoch, void *stream_)
{
    if (!c || !c->d_slot_stats) return TFE_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (freq_last && c->cfg.gpu_slots > 0)
        CU(cudaMemcpyAsync(freq_last, c->d_slot_stats, (size_t)c->cfg.gpu_slots * sizeof(uint2), cudaMemcpyDeviceToHost,
                           stream));
    if (epoch) CU(cudaMemcpyAsync(epoch, c->d_epoch, sizeof(uint32_t), cudaMemcpyDeviceToHost, stream));
    CU(cudaStreamSynchronize(stream));
    if (freq_last)                          // the device marks a slot without owner in its freq word; it has served nothing
        for (int64_t i = 0; i < c->cfg.gpu_slots; ++i)
            if (freq_last[2 * i] == TFE_FREE_SLOT_FREQ) freq_last[2 * i] = 0u;
    return TFE_OK;
}

tfe_status tfe_prefetch_candidates(tfe_ctx *c, const int32_t *history, int32_t B, int32_t H,
                                   const int32_t *cand_tokens, const float *cand_prob, int32_t K,
                                   const float *usefulness, const tfe_prefetch_params *prm,
                                   uint32_t *out_phrase, uint8_t *out_tier, float *out_score, uint32_t *out_src,
                                   uint32_t *out_count, void *stream_)
{
    if (!c || !prm || B < 0 || H < 0 || K < 0) return TFE_ERR_INVALID_ARG;
    if (prm->budget < 0 || prm->budget > TFE_PREFETCH_MAX_BUDGET) return TFE_ERR_INVALID_ARG;
    if (!(prm->benefit_host >= 0.f) || !(prm->benefit_ssd >= 0.f)) return TFE_ERR_INVALID_ARG;
    if (!out_count || (prm->budget > 0 && (!out_phrase || !out_tier || !out_score || !out_src)))
        return TFE_ERR_INVALID_ARG;
    const int64_t E = (int64_t)B * K * c->cfg.n_orders;
    if (E > 0x7FFFFFFFll) return TFE_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (E == 0) {
        CU(cudaMemsetAsync(out_count, 0, 2 * sizeof(uint32_t), stream));
        return TFE_OK;
    }
    if (!cand_tokens || !cand_prob || (H > 0 && !history)) return TFE_ERR_INVALID_ARG;
    if (E > c->pf_cap) {        // grows outside the steady state
        CU(cudaDeviceSynchronize());
        free_dev(c->d_pf_keys); free_dev(c->d_pf_phrase); free_dev(c->d_pf_tier);
        c->d_pf_keys = nullptr; c->d_pf_phrase = nullptr; c->d_pf_tier = nullptr;
        c->pf_cap = 0;
        const int64_t cap = std::max<int64_t>(E, 4096);
        CU(cudaMalloc(&c->d_pf_keys, (size_t)cap * 8));
        CU(cudaMalloc(&c->d_pf_phrase, (size_t)cap * 4));
        CU(cudaMalloc(&c->d_pf_tier, (size_t)cap));
        if (!c->d_pf_counter) {
            CU(cudaMalloc(&c->d_pf_counter, sizeof(uint32_t)));
            CU(cudaMemset(c->d_pf_counter, 0, sizeof(uint32_t)));
        }
        c->pf_cap = cap;
    }
    TfePrefetchParams p{};
    p.history = history; p.cand = cand_tokens; p.prob = cand_prob; p.usefulness = usefulness;
    p.B = B; p.H = H; p.K = K; p.n_entries = (uint32_t)E;
    p.div_orders = make_fastdiv((uint32_t)c->cfg.n_orders); p.div_k = make_fastdiv((uint32_t)K);
    p.index = c->d_index; p.n_buckets = c->n_buckets; p.phrase_tokens = c->d_phrase_tokens;
    p.n_orders = c->cfg.n_orders;
    for (int i = 0; i < 4; ++i) p.orders[i] = i < c->cfg.n_orders ? c->cfg.orders[i] : 0;
    p.tok_bits = c->tok_bits; p.vocab = c->cfg.vocab;
    p.benefit_host = prm->benefit_host; p.benefit_ssd = prm->benefit_ssd;
    p.keys = c->d_pf_keys; p.entry_phrase = c->d_pf_phrase; p.entry_tier = c->d_pf_tier; p.counter = c->d_pf_counter;
    CU(launch_overlapped(tfe_prefetch_probe_kernel, dim3((unsigned)((E + 255) / 256)), dim3(256), stream, p));
    CU(launch_overlapped(tfe_prefetch_select_kernel, dim3(1), dim3(1024), stream, c->d_pf_keys, c->d_pf_phrase, c->d_pf_tier,
                         c->d_pf_counter, (uint32_t)prm->budget, p.div_orders, (uint32_t)c->cfg.n_orders, out_phrase,
                         out_tier, out_score, out_src, out_count));
    return TFE_OK;
}

}  // extern "C"

// ---------------------------------------------------------------------------------------------
// Lookup without any allocation.
//
// tfe_lookup_inject keeps its per-call scratch (one flag byte and one phrase id per (query,
// order), plus a few counter words) in buffers the context allocates with cudaMalloc the first
// time a call needs them, and grows them when a larger call arrives.  A serving loop that has
// handed all free device memory to its own pool, or that must never hit the device-wide
// synchronisation cudaMalloc / cudaFree imply, cannot afford that.  For such callers the same
// kernels run here on a fixed scratch area that is part of the loaded library image: a file-scope
// __device__ array, present once on every GPU that loads the library, for as long as the process
// lives.  Its size bounds the call: at most TFE_NOALLOC_MAX_ENTRIES (query, order) entries.
//
// g_tfe_noalloc_scratch below is, in host code, only a handle: the kernels need the device
// address, which cudaGetSymbolAddress returns for the device that is current when it is asked.
// The first call on each device asks once and remembers the answer.
#define TFE_NOALLOC_MAX_ENTRIES 262144
#define TFE_NOALLOC_COUNTER_BYTES 256
#define TFE_NOALLOC_BYTES (TFE_NOALLOC_COUNTER_BYTES + TFE_NOALLOC_MAX_ENTRIES * 8)
static __device__ __align__(256) unsigned char g_tfe_noalloc_scratch[TFE_NOALLOC_BYTES];

namespace {
constexpr int kMaxDevices = 64;
unsigned char *g_noalloc_ptr[kMaxDevices] = {nullptr};      // device address of the array, per device
}  // namespace

extern "C" tfe_status tfe_lookup_inject_noalloc(tfe_ctx *c, const int32_t *tokens, int32_t B, int32_t T,
                                                int32_t q_start, const void *h, void *out,
                                                const tfe_inject_params *prm, uint32_t *sel_phrase,
                                                int32_t *sel_slot, uint8_t *flags, uint32_t *miss_q,
                                                uint32_t *miss_phrase, uint8_t *miss_tier, uint32_t *miss_count,
                                                void *stream_)
{
    if (!c || !prm || B < 0 || T < 0 || q_start < 0 || q_start > T) return TFE_ERR_INVALID_ARG;
    if (prm->policy != TFE_POLICY_LONGEST && prm->policy != TFE_POLICY_ALL) return TFE_ERR_INVALID_ARG;
    if (prm->gate != TFE_GATE_CONST && prm->gate != TFE_GATE_COSINE) return TFE_ERR_INVALID_ARG;
    if (!miss_q || !miss_phrase || !miss_tier || !miss_count) return TFE_ERR_INVALID_ARG;
    const int64_t Tq = T - q_start, Q = (int64_t)B * Tq;
    const int cols = prm->policy == TFE_POLICY_ALL ? c->cfg.n_orders : 1;
    if (Q * cols > TFE_NOALLOC_MAX_ENTRIES) return TFE_ERR_CAPACITY;      // the fixed scratch area is too small
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    int dev = -1;
    CU(cudaGetDevice(&dev));
    if (dev != c->device || dev < 0 || dev >= kMaxDevices) return TFE_ERR_INVALID_ARG;
    if (g_noalloc_ptr[dev] == nullptr) {       // once per device, with that device current
        void *ptr = nullptr;
        CU(cudaGetSymbolAddress(&ptr, g_tfe_noalloc_scratch));
        g_noalloc_ptr[dev] = static_cast<unsigned char *>(ptr);
    }
    unsigned char *const scratch = g_noalloc_ptr[dev];
    uint32_t *const counters = reinterpret_cast<uint32_t *>(scratch);
    if (Q != 0) {                              // a refused call leaves the shared area as it was
        if (!tokens || !h || !out) return TFE_ERR_INVALID_ARG;
        if (((reinterpret_cast<uintptr_t>(h) | reinterpret_cast<uintptr_t>(out)) & 15u) != 0)
            return TFE_ERR_INVALID_ARG;
    }
    // the area is shared by every call and keeps what the last one left: the launch state starts from zero (the
    // count of closed calls behind it, which tags the records, carries on)
    CU(cudaMemsetAsync(counters, 0, TFE_CTR_SEQ * sizeof(uint32_t), stream));
    if (Q == 0) {
        CU(cudaMemsetAsync(miss_count, 0, sizeof(uint32_t), stream));
        return TFE_OK;
    }

    uint32_t lam_bits;
    std::memcpy(&lam_bits, &prm->lambda, sizeof lam_bits);
    int variant = lookup_variant(c, prm, Q);
    if (is_longest_const(variant) && c->cfg.d / (c->cfg.hidden_dtype == 0 ? 8 : 4) >= kWideSteps) variant += kVarWide;
    int64_t qb, grid;
    lookup_geometry(c, variant, Q, &qb, &grid);
    TfeLookupParams p{};
    p.tokens = tokens; p.B = B; p.T = T; p.q_start = q_start; p.Tq = (int32_t)Tq; p.Q = (uint32_t)Q;
    p.div_tq = make_fastdiv((uint32_t)Tq); p.qb = (uint32_t)qb;
    p.q_lo = 0; p.q_hi = (uint32_t)Q; p.finalize = 1;
    p.index = c->d_index; p.n_buckets = c->n_buckets;
    p.phrase_tokens = c->d_phrase_tokens; p.rows = c->gpu_rows; p.d = c->cfg.d;
    p.h = h; p.out = out;
    p.n_orders = c->cfg.n_orders;
    for (int i = 0; i < 4; ++i) p.orders[i] = i < c->cfg.n_orders ? c->cfg.orders[i] : 0;
    p.tok_bits = c->tok_bits; p.vocab = c->cfg.vocab; p.lambda = prm->lambda;
    p.lambda_bf16x2 = (lam_bits >> 16) | (lam_bits & 0xFFFF0000u);
    p.sel_phrase = sel_phrase; p.sel_slot = sel_slot; p.flags = flags;
    p.scr_rec = reinterpret_cast<unsigned long long *>(scratch + TFE_NOALLOC_COUNTER_BYTES);
    p.miss_q = miss_q; p.miss_phrase = miss_phrase; p.miss_tier = miss_tier;
    p.counters = counters;
    pick_kernel(variant)<<<(unsigned)grid, TFE_BLOCK_THREADS, 0, stream>>>(p);
    CU(cudaGetLastError());
    CU(cudaMemcpyAsync(miss_count, counters + TFE_CTR_TOTAL, sizeof(uint32_t), cudaMemcpyDeviceToDevice, stream));
    return TFE_OK;
}
