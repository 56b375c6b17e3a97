"""Seeded synthetic inputs for the Engram lookup-and-inject path.

This module only *makes inputs* (token streams, phrase tables, residency tags,
memory rows, hidden states).  It holds none of the method's arithmetic: no key
hashing, no matching, no injection.  Both the CUDA library's tests / benchmark
and the CPU oracle's tests consume the arrays it returns; neither of those two
imports the other.

The paper builds its tables from web / encyclopedic / scientific corpora with
the backbone's tokenizer and a frozen embedding model (Sec. 4.2, Sec. 5.1);
none of those exist here, so token ids are drawn from a finite Zipf law over a
151,936-entry vocabulary, phrase tables are the de-duplicated n-gram windows of
such a stream, and rows / hidden states are synthetic numbers.

Recipe
  * Zipf sampler: P(rank r) ~ r^-s, r = 1..V, by inverse CDF.  A rank becomes a
    token id through a seeded permutation.  The table stream and the query
    filler use DIFFERENT permutations, so filler n-grams almost never occur in
    the table and the planted fraction controls the hit rate.
  * Table: every window of every configured order of the table stream, in
    stream order (by end position, then ascending order), de-duplicated on the
    exact tokens, until N entries exist.  phrase id = insertion rank.
  * Queries: filler tokens with runs copied from the table stream spliced in
    ("planting"); every window inside a planted run is a table phrase.
  * Rows / hidden states: either Gaussian numbers rounded to bf16 (small
    cases) or a counter-based procedural value s * 2^-k with s a small integer
    (exactly representable in bf16, so numpy and torch agree bit for bit),
    which lets tens of gigabytes of rows be filled on the device and looked up
    lazily on the host.
"""
from __future__ import annotations

import mmap
from dataclasses import dataclass, replace

import numpy as np

VOCAB = 151_936

# ----------------------------------------------------------------- Zipf tokens


def zipf_cdf(vocab: int, s: float) -> np.ndarray:
    w = np.arange(1, vocab + 1, dtype=np.float64) ** (-s)
    cdf = np.cumsum(w)
    return cdf / cdf[-1]


def zipf_tokens(rng: np.random.Generator, n: int, cdf: np.ndarray, perm: np.ndarray) -> np.ndarray:
    """n token ids: Zipf-distributed ranks mapped through ``perm``."""
    r = np.searchsorted(cdf, rng.random(n), side="right")
    np.minimum(r, len(cdf) - 1, out=r)
    return perm[r].astype(np.int32)


# --------------------------------------------------------------- phrase table


def _window_keys(stream: np.ndarray, n: int):
    """(hi, lo) 64-bit labels of every length-n window (21 bits per token)."""
    L = len(stream)
    s = stream.astype(np.uint64)
    m = min(n, 3)
    lo = np.zeros(L - n + 1, dtype=np.uint64)
    for k in range(m):                      # the last min(n,3) tokens
        lo = (lo << np.uint64(21)) | s[n - m + k: L - m + k + 1]
    hi = s[: L - n + 1].copy() if n == 4 else None
    return hi, lo


def _first_and_count(hi, lo):
    """Per distinct label: index of its first window and its number of windows."""
    if hi is None:
        _, first, cnt = np.unique(lo, return_index=True, return_counts=True)
        return first, cnt
    order = np.lexsort((lo, hi))            # stable: equal labels keep stream order
    shi, slo = hi[order], lo[order]
    new = np.ones(len(order), dtype=bool)
    new[1:] = (shi[1:] != shi[:-1]) | (slo[1:] != slo[:-1])
    starts = np.nonzero(new)[0]
    return order[starts], np.diff(np.append(starts, len(order)))


@dataclass
class Table:
    phrase_tokens: np.ndarray   # int32 [N,4], unused = -1
    phrase_len: np.ndarray      # uint8 [N]
    count: np.ndarray           # int64 [N] occurrences in the table stream
    stream: np.ndarray          # int32 table stream S
    safe_len: int               # every window of every order inside S[0:safe_len) is a phrase
    init_slot: np.ndarray = None   # int32 [N]: >=0 GPU slot, -1 host, -2 SSD
    gpu_slots: int = 0


def build_table(seed: int, n_phrases: int, orders, s: float, vocab: int = VOCAB) -> Table:
    perm_table = np.random.default_rng([seed, 2]).permutation(vocab)
    cdf = zipf_cdf(vocab, s)
    orders = sorted(int(o) for o in orders)
    if n_phrases > sum(min(vocab ** n, 2 ** 62) for n in orders):
        raise ValueError(f"{n_phrases} distinct phrases of orders {orders} do not exist over {vocab} token ids")
    L = max(64, int(n_phrases * 0.55) + 16)
    while True:
        S = zipf_tokens(np.random.default_rng([seed, 1]), L, cdf, perm_table)
        ends, lens, starts, cnts = [], [], [], []
        for n in orders:
            first, cnt = _first_and_count(*_window_keys(S, n))
            ends.append(first + n - 1)
            lens.append(np.full(len(first), n, dtype=np.int64))
            starts.append(first)
            cnts.append(cnt)
        ends, lens = np.concatenate(ends), np.concatenate(lens)
        starts, cnts = np.concatenate(starts), np.concatenate(cnts)
        if len(ends) >= n_phrases:
            break
        L = int(L * 1.7)
    order = np.argsort(ends * 8 + lens, kind="stable")[:n_phrases]
    ends, lens, starts, cnts = ends[order], lens[order], starts[order], cnts[order]
    pt = np.full((n_phrases, 4), -1, dtype=np.int32)
    for k in range(4):
        sel = lens > k
        pt[sel, k] = S[starts[sel] + k]
    safe_len = int(ends[-1])            # windows ending before the last inserted end are all present
    return Table(pt, lens.astype(np.uint8), cnts.astype(np.int64), S, safe_len)


def assign_residency(table: Table, seed: int, gpu_slots: int, mode: str,
                     reserve_free: int = 0) -> Table:
    """Fill ``init_slot``.

    mode "all":      every phrase GPU-resident, slot = seeded permutation of id.
    mode "hot_host": the (gpu_slots - reserve_free) phrases with the highest stream
                     count (ties: lower id) are GPU-resident in permuted slots
                     [0, gpu_slots - reserve_free); the rest are host-resident.
    mode "hot_host_ssd": as above, the rest alternate host / SSD by id parity.
    """
    N = len(table.phrase_len)
    rng = np.random.default_rng([seed, 3])
    slot = np.empty(N, dtype=np.int32)
    if mode == "all":
        assert gpu_slots >= N
        slot[:] = rng.permutation(gpu_slots)[:N].astype(np.int32)
    else:
        n_res = min(N, gpu_slots - reserve_free)
        hot = np.lexsort((np.arange(N), -table.count))[:n_res]
        slot[:] = -1
        if mode == "hot_host_ssd":
            slot[(np.arange(N) & 1) == 1] = -2
        slot[hot] = rng.permutation(n_res).astype(np.int32)
    return replace(table, init_slot=slot, gpu_slots=int(gpu_slots))


# -------------------------------------------------------------------- queries


def prefill_queries(table: Table, seed: int, B: int, T: int, p: float, s: float,
                    vocab: int = VOCAB, run_len: int = 6, variant: int = 0) -> np.ndarray:
    """int32 [B,T]: filler with planted runs; round(p*B*T) positions sit at offset >= 1 of a run."""
    rng = np.random.default_rng([seed, 5, variant])
    cdf = zipf_cdf(vocab, s)
    perm_query = np.random.default_rng([seed, 4]).permutation(vocab)
    tok = zipf_tokens(rng, B * T, cdf, perm_query).reshape(B, T)
    target = int(round(p * B * T))
    per = run_len - 1
    n_full, rem = divmod(target, per)
    runs = [run_len] * n_full + ([rem + 1] if rem else [])
    cell = run_len + 1
    cells_per_seq = T // cell
    assert len(runs) <= B * cells_per_seq, "planted fraction too high for this shape"
    assert table.safe_len > run_len + 1
    chosen = rng.choice(B * cells_per_seq, size=len(runs), replace=False)
    src = rng.integers(0, table.safe_len - run_len, size=len(runs))
    jitter = rng.integers(0, cell - run_len + 1, size=len(runs))
    for c, r, s0, j in zip(chosen, runs, src, jitter):
        b, k = divmod(int(c), cells_per_seq)
        t0 = k * cell + int(j)
        tok[b, t0:t0 + r] = table.stream[s0:s0 + r]
    return np.ascontiguousarray(tok)


def decode_queries(table: Table, seed: int, B: int, orders, p: float, s: float,
                   vocab: int = VOCAB, variant: int = 0, uniform_over_phrases: bool = False):
    """int32 [B, n_max] windows, query = last position (q_start = n_max - 1).

    Exactly round(p*B) sequences end in a planted phrase of an order drawn
    uniformly from ``orders``: copied from a uniformly chosen stream position,
    or (``uniform_over_phrases``) a uniformly chosen phrase id -- the cold-cache case.
    """
    rng = np.random.default_rng([seed, 6, variant])
    orders = sorted(int(o) for o in orders)
    n_max = orders[-1]
    cdf = zipf_cdf(vocab, s)
    perm_query = np.random.default_rng([seed, 4]).permutation(vocab)
    tok = zipf_tokens(rng, B * n_max, cdf, perm_query).reshape(B, n_max)
    n_plant = int(round(p * B))
    seqs = rng.choice(B, size=n_plant, replace=False)
    if uniform_over_phrases:
        ids = rng.integers(0, len(table.phrase_len), size=n_plant)
        for b, i in zip(seqs, ids):
            L = int(table.phrase_len[i])
            tok[b, n_max - L:] = table.phrase_tokens[i, :L]
    else:
        ell = rng.choice(np.asarray(orders), size=n_plant)
        src = rng.integers(0, table.safe_len - n_max, size=n_plant)
        for b, L, s0 in zip(seqs, ell, src):
            tok[b, n_max - L:] = table.stream[s0:s0 + L]
    return np.ascontiguousarray(tok)


# -------------------------------------------------- floating-point payloads


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even float32 -> bf16 bit patterns (input generation only)."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    u = u + np.uint64(0x7FFF) + ((u >> np.uint64(16)) & np.uint64(1))
    return (u >> np.uint64(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def gaussian_bf16(seed_seq, shape, sigma: float) -> np.ndarray:
    rng = np.random.default_rng(seed_seq)
    return f32_to_bf16_bits((rng.standard_normal(shape, dtype=np.float32) * np.float32(sigma)))


_M1 = 0xBF58476D1CE4E5B9
_M2 = 0x94D049BB133111EB
_GOLD = 0x9E3779B97F4A7C15


def _i64(c: int) -> int:
    c &= (1 << 64) - 1
    return c - (1 << 64) if c >= (1 << 63) else c


def _lsr(z, k: int):
    return (z >> k) & ((1 << (64 - k)) - 1)


def procedural_int(idx, tag: int):
    """Counter-based small integer in [-126, 126] for every int64 counter in ``idx``.

    ``idx`` is a numpy int64 array or a torch int64 tensor; the same integer
    operations (wrapping multiply, xor, logical shift) run on either, so host
    and device produce identical values.  The mixing steps are the published
    splitmix64 finaliser; the value is the centred sum of four 6-bit lanes
    (bell-shaped, standard deviation about 36.9).
    """
    z = idx ^ _i64(tag * _GOLD)
    z = (z ^ _lsr(z, 30)) * _i64(_M1)
    z = (z ^ _lsr(z, 27)) * _i64(_M2)
    z = z ^ _lsr(z, 31)
    return (z & 63) + (_lsr(z, 16) & 63) + (_lsr(z, 32) & 63) + (_lsr(z, 48) & 63) - 126


ROW_TAG, ROW_SHIFT = 0x0A11CE, 10      # rows:   s * 2^-10, std about 0.036
HID_TAG, HID_SHIFT = 0x0B0B00, 5       # hidden: s * 2^-5,  std about 1.15
HEAD_W_TAG, HEAD_W_SHIFT = 0x0EAD00, 10 # early-exit head projection rows: std about 0.036
HEAD_H_TAG, HEAD_H_SHIFT = 0x0EAD01, 5  # intermediate hidden states: std about 1.15 (logits: std about 1.3 at d = 1024)


def procedural_bf16_np(ids: np.ndarray, d: int, tag: int, shift: int) -> np.ndarray:
    """uint16 [len(ids), d] bf16 bit patterns of row ``id`` (exact, no rounding)."""
    ids = np.asarray(ids, dtype=np.int64)
    idx = ids[:, None] * d + np.arange(d, dtype=np.int64)[None, :]
    with np.errstate(over="ignore"):
        v = procedural_int(idx, tag)
    f = v.astype(np.float32) * np.float32(2.0 ** -shift)
    return (f.view(np.uint32) >> np.uint32(16)).astype(np.uint16)


def procedural_bf16_torch(ids, d: int, tag: int, shift: int):
    """torch.bfloat16 [len(ids), d] on ids.device; bit-identical to the numpy version."""
    import torch
    idx = ids.to(torch.int64)[:, None] * d + torch.arange(d, dtype=torch.int64, device=ids.device)[None, :]
    v = procedural_int(idx, tag)
    return (v.to(torch.float32) * (2.0 ** -shift)).to(torch.bfloat16)


def fill_rows_torch(rows, slot_owner, tag: int = ROW_TAG, shift: int = ROW_SHIFT,
                    chunk_rows: int = 1 << 16) -> None:
    """rows[slot] <- procedural row of phrase slot_owner[slot] (zeros where owner < 0)."""
    import torch
    C, d = rows.shape
    for s0 in range(0, C, chunk_rows):
        own = slot_owner[s0:s0 + chunk_rows]
        blk = procedural_bf16_torch(torch.clamp(own, min=0), d, tag, shift)
        blk[own < 0] = 0
        rows[s0:s0 + len(own)] = blk


class SparseRows:
    """A [C, d] uint16 array over a lazily committed anonymous mapping.

    Lets the oracle address a table of tens of gigabytes with its plain
    ``rows[slot][j]`` indexing while only the referenced rows ever get pages.
    """

    def __init__(self, C: int, d: int):
        self.nbytes = max(mmap.PAGESIZE, C * d * 2)
        self._mm = mmap.mmap(-1, self.nbytes, flags=mmap.MAP_PRIVATE | mmap.MAP_ANONYMOUS | 0x4000)  # MAP_NORESERVE
        self.array = np.frombuffer(self._mm, dtype=np.uint16, count=C * d).reshape(C, d)

    def materialise(self, slots: np.ndarray, owner_ids: np.ndarray, tag=ROW_TAG, shift=ROW_SHIFT):
        slots = np.asarray(slots, dtype=np.int64)
        if len(slots):
            self.array[slots] = procedural_bf16_np(owner_ids, self.array.shape[1], tag, shift)


# ------------------------------------------------------------------ workloads


@dataclass(frozen=True)
class Workload:
    name: str
    seed: int
    shape: str            # "prefill" | "decode"
    B: int
    T: int                # prefill: sequence length; decode: n_max
    orders: tuple
    n_phrases: int
    gpu_slots: int
    d: int = 1024
    s: float = 1.1
    p: float = 0.5
    load_factor: float = 0.7
    residency: str = "all"
    reserve_free: int = 0
    rows: str = "procedural"   # "gaussian" | "procedural"
    vocab: int = VOCAB
    note: str = ""

    @property
    def q_start(self) -> int:
        return 0 if self.shape == "prefill" else self.T - 1

    @property
    def Q(self) -> int:
        return self.B * (self.T - self.q_start)


def config(i: int, **over) -> Workload:
    """The five benchmark configurations (index 1..5), overridable for scaled-down cases."""
    base = {
        1: Workload("c1_tiny", 0, "prefill", 4, 16, (2, 3), 20_000, 20_000, p=0.5, rows="gaussian"),
        2: Workload("c2_decode64", 2, "decode", 64, 3, (2, 3), 1_000_000, 262_144, p=0.6,
                    residency="hot_host"),
        3: Workload("c3_prefill8x4096", 3, "prefill", 8, 4096, (2, 3, 4), 4_000_000, 4_000_000, p=0.4),
        4: Workload("c4_ssd_decode256", 4, "decode", 256, 3, (2, 3), 32_000_000, 16_777_216, s=1.2,
                    p=0.6, residency="hot_host_ssd", reserve_free=262_144),
        5: Workload("c5_sweep", 5, "decode", 65_536, 3, (2, 3), 8_000_000, 8_000_000, p=0.9),
    }[i]
    return replace(base, **over)


def make_table(w: Workload) -> Table:
    t = build_table(w.seed, w.n_phrases, w.orders, w.s, w.vocab)
    return assign_residency(t, w.seed, w.gpu_slots, w.residency, w.reserve_free)


def make_queries(w: Workload, table: Table, variant: int = 0, **kw) -> np.ndarray:
    if w.shape == "prefill":
        return prefill_queries(table, w.seed, w.B, w.T, w.p, w.s, w.vocab, variant=variant)
    return decode_queries(table, w.seed, w.B, w.orders, w.p, w.s, w.vocab, variant=variant, **kw)


def slot_owner_of(table: Table) -> np.ndarray:
    own = np.full(table.gpu_slots, -1, dtype=np.int64)
    res = np.nonzero(table.init_slot >= 0)[0]
    own[table.init_slot[res]] = res
    return own


def make_rows_np(w: Workload, table: Table) -> np.ndarray:
    """uint16 [C, d] GPU-tier rows on the host (small tables only)."""
    own = slot_owner_of(table)
    rows = np.zeros((w.gpu_slots, w.d), dtype=np.uint16)
    occ = np.nonzero(own >= 0)[0]
    if w.rows == "gaussian":
        allrows = gaussian_bf16([w.seed, 7], (w.n_phrases, w.d), 1.0 / 32.0)
        rows[occ] = allrows[own[occ]]
    else:
        rows[occ] = procedural_bf16_np(own[occ], w.d, ROW_TAG, ROW_SHIFT)
    return rows


def phrase_rows_np(w: Workload, ids: np.ndarray) -> np.ndarray:
    """uint16 [len(ids), d]: the memory vector of each phrase id (any tier)."""
    if w.rows == "gaussian":
        allrows = gaussian_bf16([w.seed, 7], (w.n_phrases, w.d), 1.0 / 32.0)
        return allrows[np.asarray(ids, dtype=np.int64)]
    return procedural_bf16_np(ids, w.d, ROW_TAG, ROW_SHIFT)


def make_hidden_np(w: Workload, variant: int = 0, Q: int | None = None) -> np.ndarray:
    """uint16 [Q, d] bf16 hidden states."""
    Q = w.Q if Q is None else Q
    if w.rows == "gaussian":
        return gaussian_bf16([w.seed, 8, variant], (Q, w.d), 1.0)
    ids = np.arange(Q, dtype=np.int64) + variant * (1 << 24)
    return procedural_bf16_np(ids, w.d, HID_TAG, HID_SHIFT)


def make_hidden_torch(w: Workload, device, variant: int = 0, Q: int | None = None):
    import torch
    Q = w.Q if Q is None else Q
    if w.rows == "gaussian":
        return torch.from_numpy(make_hidden_np(w, variant, Q).view(np.int16)).view(torch.bfloat16).to(device)
    out = torch.empty((Q, w.d), dtype=torch.bfloat16, device=device)
    step = 1 << 14
    for q0 in range(0, Q, step):
        ids = torch.arange(q0, min(Q, q0 + step), dtype=torch.int64, device=device) + variant * (1 << 24)
        out[q0:q0 + len(ids)] = procedural_bf16_torch(ids, w.d, HID_TAG, HID_SHIFT)
    return out


# ---------------------------------------------------------------- early-exit head inputs

def head_weights_np(V: int, d: int, rows=None) -> np.ndarray:
    """uint16 [V, d] (or the given rows) of the synthetic prefetch-head projection W_pref."""
    ids = np.arange(V, dtype=np.int64) if rows is None else np.asarray(rows, np.int64)
    return procedural_bf16_np(ids, d, HEAD_W_TAG, HEAD_W_SHIFT)


def head_weights_torch(V: int, d: int, device, chunk_rows: int = 1 << 15):
    import torch
    W = torch.empty((V, d), dtype=torch.bfloat16, device=device)
    for r0 in range(0, V, chunk_rows):
        r1 = min(V, r0 + chunk_rows)
        W[r0:r1] = procedural_bf16_torch(torch.arange(r0, r1, device=device), d, HEAD_W_TAG, HEAD_W_SHIFT)
    return W


def head_hidden_np(B: int, d: int, variant: int = 0) -> np.ndarray:
    return procedural_bf16_np(np.arange(B, dtype=np.int64) + variant * 100_003, d, HEAD_H_TAG, HEAD_H_SHIFT)


def head_hidden_torch(B: int, d: int, device, variant: int = 0):
    import torch
    return procedural_bf16_torch(torch.arange(B, device=device) + variant * 100_003, d, HEAD_H_TAG, HEAD_H_SHIFT)


# ------------------------------------------------------------------ corpus for n-gram extraction


def make_corpus(seed: int, L: int, vocab: int = VOCAB, *, s: float = 1.1, n_expr: int = 0, expr_rate: float = 0.3,
                expr_s: float = 1.05, doc_len: int = 512, chunk: int = 1 << 24) -> np.ndarray:
    """A tokenised corpus int32 [L] for the construction pipeline: Zipf-distributed ids (exponent ``s``, ranks
    mapped through a seeded permutation of the whole vocabulary, so ids need all their bits), with
    multi-token expressions (``n_expr`` of them, 2..4 ids each, Zipf-distributed popularity) written over
    the filler at about ``expr_rate`` of the positions, cut into documents of geometric length (mean
    ``doc_len``) by -1 separators.  Generated in chunks, reproducible for any chunk-independent prefix."""
    rng = np.random.default_rng([seed, 424242])
    perm = rng.permutation(vocab)
    cdf = zipf_cdf(vocab, s)
    n_expr = int(n_expr) if n_expr else max(16, L // 64)
    expr_len = rng.integers(2, 5, size=n_expr)
    expr_tok = zipf_tokens(rng, 4 * n_expr, cdf, perm).reshape(n_expr, 4)
    ecdf = zipf_cdf(n_expr, expr_s)
    out = np.empty(L, np.int32)
    for lo in range(0, L, chunk):
        n = min(chunk, L - lo)
        crng = np.random.default_rng([seed, 424243, lo // chunk])
        tok = zipf_tokens(crng, n, cdf, perm)
        n_starts = int(n * expr_rate / 3)
        starts = crng.integers(0, max(1, n - 4), size=n_starts)
        which = np.minimum(np.searchsorted(ecdf, crng.random(n_starts), side="right"), n_expr - 1)
        for j in range(4):
            sel = expr_len[which] > j
            tok[starts[sel] + j] = expr_tok[which[sel], j]
        n_docs = max(1, n // max(2, doc_len))
        tok[crng.integers(0, n, size=n_docs)] = -1
        out[lo:lo + n] = tok
    return out
