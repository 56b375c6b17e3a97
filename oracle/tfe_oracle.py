"""ctypes front end of the CPU oracle (``tfe_oracle.c``).

TEST INFRASTRUCTURE, NOT PRODUCT CODE: only the tests, the smoke check and the
benchmark's CPU-baseline / reference legs import this module.  It imports
nothing from the CUDA package and the CUDA package never imports it.

The front end only marshals numpy arrays; every step of the definition runs in
the C file.  ``Oracle`` bundles the table state (phrases, residency, GPU-tier
rows) so that tests read like the method: ``lookup`` = match + select + tier
walk + miss list, ``inject`` = aggregation + gated residual update,
``cache_install`` = insertion into the GPU tier.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "tfe_oracle.c")
_LIB = os.path.join(_HERE, "libtfe_oracle.so")

POLICY_LONGEST, POLICY_ALL = 0, 1
GATE_CONST, GATE_COSINE = 0, 1
HIDDEN_BF16, HIDDEN_F32 = 0, 1
ABSENT_PHRASE = 0xFFFFFFFF


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (plain C11, -O2, OpenMP when available)."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    base = ["gcc", "-O2", "-std=c11", "-D_GNU_SOURCE", "-fPIC", "-shared",
            "-ffp-contract=off", _SRC, "-lm", "-o", _LIB]
    try:
        subprocess.run(base[:1] + ["-fopenmp"] + base[1:], check=True,
                       capture_output=True, text=True)
    except subprocess.CalledProcessError:
        subprocess.run(base, check=True, capture_output=True, text=True)
    return _LIB


_lib = None


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.orc_bf16_to_double.restype = C.c_double
        _lib.orc_bf16_to_double.argtypes = [C.c_uint16]
        _lib.orc_bf16_from_double.restype = C.c_uint16
        _lib.orc_bf16_from_double.argtypes = [C.c_double]
        _lib.orc_num_threads.restype = C.c_int
        _lib.orc_sort_phrases.restype = C.c_int64
        _lib.orc_select.restype = C.c_int64
        _lib.orc_cache_install.restype = C.c_int32
        _lib.orc_cache_install_lenient.restype = C.c_int32
        _lib.orc_prefetch_candidates.restype = C.c_int64
        _lib.orc_cache_victims.restype = C.c_int64
        _lib.orc_retention_key.restype = C.c_uint32
        _lib.orc_retention_key.argtypes = [C.c_uint32, C.c_uint32, C.c_uint32, C.c_int32]
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _c(a, dtype):
    a = np.ascontiguousarray(a, dtype=dtype)
    return a


def num_threads() -> int:
    return int(lib().orc_num_threads())


def bf16_to_double(bits) -> np.ndarray:
    bits = np.asarray(bits, dtype=np.uint16)
    f = lib().orc_bf16_to_double
    return np.array([f(int(b)) for b in bits.ravel()], dtype=np.float64).reshape(bits.shape)


def bf16_from_double(x) -> np.ndarray:
    x = np.asarray(x, dtype=np.float64)
    f = lib().orc_bf16_from_double
    return np.array([f(float(v)) for v in x.ravel()], dtype=np.uint16).reshape(x.shape)


@dataclass
class LookupResult:
    match: np.ndarray        # int64 [Q, n_orders]: phrase id or -1 per order
    sel_phrase: np.ndarray   # uint32 [Q] (LONGEST) or [Q, n_orders] (ALL)
    sel_slot: np.ndarray     # int32, same shape
    flags: np.ndarray        # uint8, same shape
    miss_q: np.ndarray       # uint32 [n_miss]
    miss_phrase: np.ndarray  # uint32 [n_miss]
    miss_tier: np.ndarray    # uint8 [n_miss]


class Oracle:
    """Table state + the four operations of the path, all on the CPU."""

    def __init__(self, phrase_tokens, phrase_len, init_slot, rows, *, d, vocab, orders,
                 gpu_slots):
        self.phrase_tokens = _c(phrase_tokens, np.int32).reshape(-1, 4)
        self.phrase_len = _c(phrase_len, np.uint8)
        self.N = int(self.phrase_len.shape[0])
        self.slot_state = _c(init_slot, np.int32).copy()
        self.d, self.vocab, self.C = int(d), int(vocab), int(gpu_slots)
        self.orders = _c(orders, np.int32)
        self.rows = rows  # uint16 [C, d]; may be a sparse mapping, used in place
        self.slot_owner = np.full(self.C, -1, dtype=np.int64)
        res = np.nonzero(self.slot_state >= 0)[0]
        self.slot_owner[self.slot_state[res]] = res
        self._perm = None
        # retention state of the GPU tier (frequency, epoch of last use), epoch = lookups so far
        self.freq = np.zeros(self.C, np.uint32)
        self.last = np.zeros(self.C, np.uint32)
        self.epoch = 0

    # -- exact match ------------------------------------------------------
    def sorted_perm(self) -> np.ndarray:
        if self._perm is None:
            perm = np.empty(self.N, dtype=np.int64)
            dup = lib().orc_sort_phrases(C.c_int64(self.N), _p(self.phrase_tokens),
                                         _p(self.phrase_len), _p(perm))
            if dup:
                raise ValueError(f"{dup} duplicate phrase tuples")
            self._perm = perm
        return self._perm

    def match(self, tokens, q_start=0, matcher="sorted") -> np.ndarray:
        tokens = _c(tokens, np.int32)
        B, T = tokens.shape
        Q = B * (T - q_start)
        out = np.empty((Q, len(self.orders)), dtype=np.int64)
        common = (_p(tokens), C.c_int32(B), C.c_int32(T), C.c_int32(q_start),
                  C.c_int32(self.vocab), C.c_int32(len(self.orders)), _p(self.orders), _p(out))
        if matcher == "brute":
            lib().orc_match_brute(C.c_int64(self.N), _p(self.phrase_tokens),
                                  _p(self.phrase_len), *common)
        else:
            lib().orc_match_sorted(C.c_int64(self.N), _p(self.phrase_tokens),
                                   _p(self.phrase_len), _p(self.sorted_perm()), *common)
        return out

    # -- selection + tier walk + miss list ----------------------------------
    def select(self, match, policy=POLICY_LONGEST) -> LookupResult:
        Q, no = match.shape
        shape = (Q,) if policy == POLICY_LONGEST else (Q, no)
        sel_phrase = np.empty(shape, np.uint32)
        sel_slot = np.empty(shape, np.int32)
        flags = np.empty(shape, np.uint8)
        cap = max(1, Q * no)
        mq, mp, mt = np.empty(cap, np.uint32), np.empty(cap, np.uint32), np.empty(cap, np.uint8)
        n = lib().orc_select(C.c_int32(policy), C.c_int64(Q), C.c_int32(no), _p(match),
                             _p(self.slot_state), _p(sel_phrase), _p(sel_slot), _p(flags),
                             _p(mq), _p(mp), _p(mt))
        return LookupResult(match, sel_phrase, sel_slot, flags, mq[:n].copy(), mp[:n].copy(),
                            mt[:n].copy())

    def lookup(self, tokens, q_start=0, policy=POLICY_LONGEST, matcher="sorted") -> LookupResult:
        return self.select(self.match(tokens, q_start, matcher), policy)

    # -- aggregation + gated residual injection -----------------------------
    def inject(self, res: LookupResult, h, *, policy=POLICY_LONGEST, gate=GATE_CONST, lam=1.0,
               hidden_dtype=HIDDEN_BF16, want_exact=True):
        """Returns (out_exact float64 [Q,d] or None, out_rounded in the hidden dtype)."""
        h = _c(h, np.float32 if hidden_dtype == HIDDEN_F32 else np.uint16)
        Q = res.match.shape[0]
        assert h.shape == (Q, self.d)
        exact = np.empty((Q, self.d), np.float64) if want_exact else None
        rounded = np.empty_like(h)
        lib().orc_inject(C.c_int32(policy), C.c_int32(gate), C.c_double(lam), C.c_int64(Q),
                         C.c_int32(self.d), C.c_int32(len(self.orders)), _p(self.orders),
                         _p(res.sel_slot), _p(res.flags), _p(self.rows), _p(h),
                         C.c_int32(hidden_dtype), _p(exact), _p(rounded))
        return exact, rounded

    # -- GPU-tier installation ------------------------------------------------
    def cache_install(self, ids, src_rows, dst_slots) -> int:
        ids = _c(ids, np.uint32)
        dst = _c(dst_slots, np.int32)
        src = None if src_rows is None else _c(src_rows, np.uint16)
        rc = int(lib().orc_cache_install(
            C.c_int64(self.N), C.c_int64(self.C), C.c_int32(self.d), _p(self.slot_state),
            _p(self.slot_owner), _p(self.rows), C.c_int32(len(ids)), _p(ids), _p(src), _p(dst)))
        if rc == 0:
            lib().orc_cache_installed(C.c_int32(len(ids)), _p(dst), C.c_uint32(self.epoch), _p(self.freq),
                                      _p(self.last))
        return rc

    def cache_install_lenient(self, ids, src_rows, dst_slots):
        """Skips what cannot be applied; returns (applied uint8 [n], count)."""
        ids = _c(ids, np.uint32)
        dst = _c(dst_slots, np.int32)
        src = None if src_rows is None else _c(src_rows, np.uint16)
        applied = np.zeros(max(len(ids), 1), np.uint8)
        cnt = int(lib().orc_cache_install_lenient(
            C.c_int64(self.N), C.c_int64(self.C), C.c_int32(self.d), _p(self.slot_state), _p(self.slot_owner),
            _p(self.rows), C.c_int32(len(ids)), _p(ids), _p(src), _p(dst), _p(applied)))
        applied = applied[:len(ids)]
        if cnt:
            done = _c(dst[applied == 1], np.int32)
            lib().orc_cache_installed(C.c_int32(len(done)), _p(done), C.c_uint32(self.epoch), _p(self.freq),
                                      _p(self.last))
        return applied, cnt

    # -- GPU-tier retention ranking ---------------------------------------------
    def touch(self, res: LookupResult) -> None:
        """Account one lookup call: bump the slots it injected from, then advance the epoch."""
        flags = _c(res.flags, np.uint8).ravel()
        slots = _c(res.sel_slot, np.int32).ravel()
        lib().orc_cache_touch(C.c_int64(flags.size), _p(flags), _p(slots), C.c_uint32(self.epoch),
                              _p(self.freq), _p(self.last))
        self.epoch += 1

    def cache_victims(self, n, half_life=0):
        """(slots int32[m], keys uint32[m]), m = min(n, C): ascending (retention key, slot)."""
        m = min(int(n), self.C)
        slots, keys = np.empty(max(m, 1), np.int32), np.empty(max(m, 1), np.uint32)
        got = lib().orc_cache_victims(C.c_int64(self.C), _p(self.slot_owner), _p(self.freq), _p(self.last),
                                      C.c_uint32(self.epoch), C.c_int32(half_life), C.c_int64(n), _p(slots),
                                      _p(keys))
        return slots[:got].copy(), keys[:got].copy()

    # -- prefetch candidates + priority ------------------------------------------
    def prefetch_candidates(self, history, cand, prob, *, usefulness=None, benefit_host=1.0, benefit_ssd=2.0,
                            budget=4096):
        """(phrase uint32[n], tier uint8[n], score float32[n], src uint32[n], total candidates)."""
        history = _c(history, np.int32)
        cand = _c(cand, np.int32)
        prob = _c(prob, np.float32)
        B, H = history.shape
        K = cand.shape[1]
        use = None if usefulness is None else _c(usefulness, np.float32)
        op, ot = np.empty(max(budget, 1), np.uint32), np.empty(max(budget, 1), np.uint8)
        osc, osr = np.empty(max(budget, 1), np.float32), np.empty(max(budget, 1), np.uint32)
        total = lib().orc_prefetch_candidates(
            C.c_int64(self.N), _p(self.phrase_tokens), _p(self.phrase_len), _p(self.sorted_perm()),
            _p(self.slot_state), _p(history), C.c_int32(B), C.c_int32(H), _p(cand), _p(prob), C.c_int32(K),
            C.c_int32(self.vocab), C.c_int32(len(self.orders)), _p(self.orders), _p(use),
            C.c_float(benefit_host), C.c_float(benefit_ssd), C.c_int32(budget), _p(op), _p(ot), _p(osc), _p(osr))
        n = int(min(total, budget))
        return op[:n].copy(), ot[:n].copy(), osc[:n].copy(), osr[:n].copy(), int(total)


# -- early-exit prefetch head (independent of any phrase table) ---------------------------------
def head_logits(W, h) -> np.ndarray:
    """float64 [B, V]: W_pref h for bf16 bit patterns W [V, d], h [B, d]."""
    W, h = _c(W, np.uint16), _c(h, np.uint16)
    V, d = W.shape
    B = h.shape[0]
    assert h.shape[1] == d
    z = np.empty((B, V), np.float64)
    lib().orc_head_logits(C.c_int32(V), C.c_int32(d), C.c_int32(B), _p(W), _p(h), _p(z))
    return z


def head_topk(z, K):
    """(tokens int32 [B, K], prob float64 [B, K], lse float64 [B]) of softmax over each row of z."""
    z = _c(z, np.float64)
    B, V = z.shape
    tokens, prob, lse = np.empty((B, K), np.int32), np.empty((B, K), np.float64), np.empty(B, np.float64)
    lib().orc_head_topk(C.c_int32(V), C.c_int32(B), C.c_int32(K), _p(z), _p(tokens), _p(prob), _p(lse))
    return tokens, prob, lse


# -- n-gram extraction with a frequency threshold (independent of any phrase table) ---------------
def mine_ngrams(tokens, vocab, orders, min_count=1, cap=None, hist_bins=1024):
    """(phrase_tokens int32 [n, 4], phrase_len uint8 [n], count uint32 [n], n_found, distinct int64
    [n_orders], hist int64 [hist_bins]); n = min(n_found, cap), ascending (first occurrence, order)."""
    tokens = _c(tokens, np.int32).reshape(-1)
    orders = _c(orders, np.int32)
    L = len(tokens)
    cap = L * len(orders) if cap is None else int(cap)
    pt = np.full((max(cap, 1), 4), -1, np.int32)
    pl, pc = np.zeros(max(cap, 1), np.uint8), np.zeros(max(cap, 1), np.uint32)
    distinct, hist = np.zeros(len(orders), np.int64), np.zeros(hist_bins, np.int64)
    f = lib().orc_mine_ngrams
    f.restype = C.c_int64
    n_found = f(C.c_int64(L), _p(tokens), C.c_int32(vocab), C.c_int32(len(orders)), _p(orders),
                C.c_uint32(min_count), C.c_int64(cap), _p(pt), _p(pl), _p(pc), _p(distinct),
                C.c_int32(hist_bins), _p(hist))
    n = int(min(n_found, cap))
    return pt[:n].copy(), pl[:n].copy(), pc[:n].copy(), int(n_found), distinct, hist


def count_tuple(tokens, tup):
    """(count, first end position or -1) of one tuple of valid ids in the corpus."""
    tokens = _c(tokens, np.int32).reshape(-1)
    tup = _c(tup, np.int32)
    first = C.c_int64(-1)
    f = lib().orc_count_tuple
    f.restype = C.c_int64
    n = f(C.c_int64(len(tokens)), _p(tokens), C.c_int32(len(tup)), _p(tup), C.byref(first))
    return int(n), int(first.value)


def assign_residency(count, gpu_slots, host_min_count=2):
    """(init_slot int32 [N], (n_gpu, n_host, n_ssd)): the gpu_slots most frequent phrases in the GPU tier."""
    count = _c(count, np.uint32)
    N = len(count)
    init_slot, tiers = np.empty(max(N, 1), np.int32), np.zeros(3, np.int64)
    lib().orc_assign_residency(C.c_int64(N), _p(count), C.c_int64(gpu_slots), C.c_uint32(host_min_count),
                               _p(init_slot), _p(tiers))
    return init_slot[:N].copy(), tuple(int(x) for x in tiers)
