"""ctypes binding of libtfe.so: the same entry points as include/tfe.h.

Argument marshalling only -- every step of the path runs in the library's CUDA
kernels.  Device buffers are ``torch`` CUDA tensors (or raw integer addresses);
host buffers are numpy arrays or pinned CPU tensors.  Loading fails loudly when
the shared library has not been built; there is no CPU fallback.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("TFE_LIB") or os.path.join(_HERE, "libtfe.so")   # TFE_LIB: a tuning build

TFE_OK = 0
STATUS_NAMES = ["TFE_OK", "TFE_ERR_INVALID_ARG", "TFE_ERR_DUPLICATE_PHRASE", "TFE_ERR_KEY_COLLISION",
                "TFE_ERR_CAPACITY", "TFE_ERR_SLOT_RANGE", "TFE_ERR_UNKNOWN_PHRASE",
                "TFE_ERR_ALREADY_RESIDENT", "TFE_ERR_MISS_OVERFLOW", "TFE_ERR_PROBE_LIMIT",
                "TFE_ERR_CUDA", "TFE_ERR_INTERNAL"]
(TFE_ERR_INVALID_ARG, TFE_ERR_DUPLICATE_PHRASE, TFE_ERR_KEY_COLLISION, TFE_ERR_CAPACITY,
 TFE_ERR_SLOT_RANGE, TFE_ERR_UNKNOWN_PHRASE, TFE_ERR_ALREADY_RESIDENT, TFE_ERR_MISS_OVERFLOW,
 TFE_ERR_PROBE_LIMIT, TFE_ERR_CUDA, TFE_ERR_INTERNAL) = range(1, 12)
POLICY_LONGEST, POLICY_ALL = 0, 1
GATE_CONST, GATE_COSINE = 0, 1
HIDDEN_BF16, HIDDEN_F32 = 0, 1
NO_PHRASE = 0xFFFFFFFF

EXPORTS = ["tfe_index_build", "tfe_index_build_device", "tfe_cache_install", "tfe_cache_install_device", "tfe_lookup_inject", "tfe_lookup_inject_host",
           "tfe_miss_list", "tfe_miss_list_device", "tfe_destroy", "tfe_status_string",
           "tfe_last_cuda_error", "tfe_index_geometry", "tfe_phrase_key64", "tfe_home_bucket",
           "tfe_launch_geometry", "tfe_set_tuning", "tfe_lookup_inject_noalloc", "tfe_prefetch_candidates",
           "tfe_cache_policy_enable", "tfe_cache_select_victims", "tfe_cache_select_victims_device",
           "tfe_cache_stats", "tfe_head_create", "tfe_head_destroy", "tfe_head_topk", "tfe_head_buffers",
           "tfe_head_status", "tfe_head_geometry", "tfe_mine_ngrams", "tfe_mine_workspace_bytes", "tfe_assign_residency", "tfe_stream_copy",
           "tfe_cache_select_tuning"]


class TfeConfig(C.Structure):
    _fields_ = [("d", C.c_int32), ("vocab", C.c_int32), ("n_orders", C.c_int32),
                ("orders", C.c_int32 * 4), ("n_phrases", C.c_int64), ("gpu_slots", C.c_int64),
                ("load_factor", C.c_float), ("hidden_dtype", C.c_int32),
                ("max_kicks", C.c_int32)]


class TfeInjectParams(C.Structure):
    _fields_ = [("policy", C.c_int32), ("gate", C.c_int32), ("lam", C.c_float)]


class TfePrefetchParams(C.Structure):
    _fields_ = [("benefit_host", C.c_float), ("benefit_ssd", C.c_float), ("budget", C.c_int32)]


class TfeError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        detail = ""
        if status == TFE_ERR_CUDA:
            detail = ": " + lib().tfe_last_cuda_error().decode()
        super().__init__(f"{where}: {STATUS_NAMES[status]} ({lib().tfe_status_string(status).decode()}){detail}")


_lib = None


def lib() -> C.CDLL:
    """The loaded library.  Raises if it is not built: this package has no other compute path."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with "
                               "`python -m paper_2607_07388_b200.build` (needs nvcc); there is no fallback")
        L = C.CDLL(LIB_PATH)
        vp, i32, i64, u64 = C.c_void_p, C.c_int32, C.c_int64, C.c_uint64
        L.tfe_index_build.argtypes = [C.POINTER(TfeConfig), vp, vp, vp, vp, vp, C.POINTER(vp)]
        L.tfe_index_build_device.argtypes = L.tfe_index_build.argtypes
        L.tfe_cache_install.argtypes = [vp, i32, vp, vp, vp, vp]
        L.tfe_cache_install_device.argtypes = [vp, i32, vp, vp, vp, vp, vp, vp]
        L.tfe_lookup_inject.argtypes = [vp, vp, i32, i32, i32, vp, vp, C.POINTER(TfeInjectParams), vp, vp, vp, vp]
        L.tfe_lookup_inject_host.argtypes = L.tfe_lookup_inject.argtypes
        L.tfe_lookup_inject_noalloc.argtypes = [vp, vp, i32, i32, i32, vp, vp, C.POINTER(TfeInjectParams), vp, vp, vp,
                                                vp, vp, vp, vp, vp]
        L.tfe_miss_list.argtypes = [vp, vp, vp, vp, i64, C.POINTER(i64), vp]
        L.tfe_prefetch_candidates.argtypes = [vp, vp, i32, i32, vp, vp, i32, vp, C.POINTER(TfePrefetchParams),
                                              vp, vp, vp, vp, vp, vp]
        L.tfe_miss_list_device.argtypes = [vp, C.POINTER(vp), C.POINTER(vp), C.POINTER(vp), C.POINTER(vp)]
        L.tfe_destroy.argtypes = [vp]
        L.tfe_destroy.restype = None
        L.tfe_status_string.argtypes = [C.c_int]
        L.tfe_status_string.restype = C.c_char_p
        L.tfe_last_cuda_error.restype = C.c_char_p
        L.tfe_index_geometry.argtypes = [vp, C.POINTER(i64), C.POINTER(i64), C.POINTER(i64)]
        L.tfe_phrase_key64.argtypes = [i32, vp, i32, C.POINTER(i32)]
        L.tfe_phrase_key64.restype = u64
        L.tfe_home_bucket.argtypes = [u64, u64]
        L.tfe_home_bucket.restype = u64
        L.tfe_launch_geometry.argtypes = [vp, C.POINTER(i32), C.POINTER(i32), C.POINTER(i32)]
        L.tfe_set_tuning.argtypes = [vp, i32]
        L.tfe_cache_policy_enable.argtypes = [vp, vp]
        L.tfe_cache_select_victims.argtypes = [vp, i32, i32, vp, vp, C.POINTER(i32), vp]
        L.tfe_cache_select_victims_device.argtypes = [vp, C.POINTER(vp), C.POINTER(vp)]
        L.tfe_cache_stats.argtypes = [vp, vp, C.POINTER(C.c_uint32), vp]
        L.tfe_head_create.argtypes = [vp, i32, i32, i32, C.POINTER(vp)]
        L.tfe_head_destroy.argtypes = [vp]
        L.tfe_head_destroy.restype = None
        L.tfe_head_topk.argtypes = [vp, vp, i32, i32, vp, vp, vp]
        L.tfe_head_buffers.argtypes = [vp, C.POINTER(vp), C.POINTER(i64), C.POINTER(vp)]
        L.tfe_head_status.argtypes = [vp, C.POINTER(C.c_uint32), vp]
        L.tfe_head_geometry.argtypes = [vp, C.POINTER(i32), C.POINTER(i32), C.POINTER(i32)]
        L.tfe_mine_ngrams.argtypes = [vp, i64, i32, i32, vp, C.c_uint32, i64, vp, vp, vp, C.POINTER(i64), vp, vp, vp, i64, vp]
        L.tfe_mine_workspace_bytes.argtypes = [i64, i32]
        L.tfe_assign_residency.argtypes = [vp, i64, i64, C.c_uint32, vp, vp, vp]
        L.tfe_mine_workspace_bytes.restype = i64
        L.tfe_stream_copy.argtypes = [vp, vp, i64, vp]
        L.tfe_cache_select_tuning.argtypes = [vp, i32, i32, i32]
        for name in ("tfe_index_build", "tfe_index_build_device", "tfe_cache_install", "tfe_cache_install_device", "tfe_lookup_inject", "tfe_lookup_inject_host",
                     "tfe_miss_list", "tfe_miss_list_device", "tfe_index_geometry", "tfe_launch_geometry",
                     "tfe_set_tuning", "tfe_lookup_inject_noalloc", "tfe_prefetch_candidates",
                     "tfe_cache_policy_enable", "tfe_cache_select_victims", "tfe_cache_select_victims_device",
                     "tfe_cache_stats", "tfe_head_create", "tfe_head_topk", "tfe_head_buffers", "tfe_head_status",
                     "tfe_head_geometry", "tfe_mine_ngrams", "tfe_assign_residency", "tfe_cache_select_tuning"):
            getattr(L, name).restype = C.c_int
        _lib = L
    return _lib


def _addr(x):
    """Address of a device tensor, host tensor, numpy array, int or None."""
    if x is None:
        return None
    if isinstance(x, int):
        return x
    if isinstance(x, np.ndarray):
        assert x.flags["C_CONTIGUOUS"]
        return x.ctypes.data
    assert x.is_contiguous()
    return x.data_ptr()


def _stream(stream):
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    return stream if isinstance(stream, int) else stream.cuda_stream


def _check(status: int, where: str):
    if status != TFE_OK:
        raise TfeError(status, where)


def make_config(*, d, vocab, orders, n_phrases, gpu_slots, load_factor=0.7, hidden_dtype=HIDDEN_BF16,
                max_kicks=0) -> TfeConfig:
    cfg = TfeConfig()
    cfg.d, cfg.vocab, cfg.n_orders = int(d), int(vocab), len(orders)
    for i in range(4):
        cfg.orders[i] = int(orders[i]) if i < len(orders) else 0
    cfg.n_phrases, cfg.gpu_slots = int(n_phrases), int(gpu_slots)
    cfg.load_factor, cfg.hidden_dtype, cfg.max_kicks = float(load_factor), int(hidden_dtype), int(max_kicks)
    return cfg


# ---- the C entry points, same names -------------------------------------------------------


def tfe_index_build(cfg: TfeConfig, phrase_tokens, phrase_len, init_slot, gpu_rows, stream=None) -> int:
    """Returns the context handle (an integer address)."""
    pt = np.ascontiguousarray(phrase_tokens, dtype=np.int32)
    pl = np.ascontiguousarray(phrase_len, dtype=np.uint8)
    sl = np.ascontiguousarray(init_slot, dtype=np.int32)
    out = C.c_void_p()
    _check(lib().tfe_index_build(C.byref(cfg), _addr(pt), _addr(pl), _addr(sl), _addr(gpu_rows),
                                 _stream(stream), C.byref(out)), "tfe_index_build")
    return out.value


def tfe_index_build_device(cfg: TfeConfig, phrase_tokens, phrase_len, init_slot, gpu_rows, stream=None) -> int:
    """As tfe_index_build, with the three phrase arrays on the device (int32 [N,4], uint8 [N], int32 [N])."""
    out = C.c_void_p()
    _check(lib().tfe_index_build_device(C.byref(cfg), _addr(phrase_tokens), _addr(phrase_len), _addr(init_slot),
                                        _addr(gpu_rows), _stream(stream), C.byref(out)), "tfe_index_build_device")
    return out.value


def tfe_cache_install(ctx: int, phrase_ids, src_rows, dst_slots, stream=None) -> None:
    ids = np.ascontiguousarray(phrase_ids, dtype=np.uint32)
    dst = np.ascontiguousarray(dst_slots, dtype=np.int32)
    _check(lib().tfe_cache_install(ctx, len(ids), _addr(ids), _addr(src_rows), _addr(dst), _stream(stream)),
           "tfe_cache_install")


def _params(policy, gate, lam):
    p = TfeInjectParams()
    p.policy, p.gate, p.lam = int(policy), int(gate), float(lam)
    return p


def tfe_lookup_inject(ctx: int, tokens, B, T, q_start, h, out, *, policy=POLICY_LONGEST, gate=GATE_CONST,
                      lam=1.0, sel_phrase=None, sel_slot=None, flags=None, stream=None) -> None:
    p = _params(policy, gate, lam)
    _check(lib().tfe_lookup_inject(ctx, _addr(tokens), B, T, q_start, _addr(h), _addr(out), C.byref(p),
                                   _addr(sel_phrase), _addr(sel_slot), _addr(flags), _stream(stream)),
           "tfe_lookup_inject")


def tfe_lookup_inject_host(ctx: int, tokens, B, T, q_start, h, out, *, policy=POLICY_LONGEST,
                           gate=GATE_CONST, lam=1.0, sel_phrase=None, sel_slot=None, flags=None,
                           stream=None) -> None:
    p = _params(policy, gate, lam)
    _check(lib().tfe_lookup_inject_host(ctx, _addr(tokens), B, T, q_start, _addr(h), _addr(out), C.byref(p),
                                        _addr(sel_phrase), _addr(sel_slot), _addr(flags), _stream(stream)),
           "tfe_lookup_inject_host")


NOALLOC_MAX_ENTRIES = 262_144


def tfe_lookup_inject_noalloc(ctx: int, tokens, B, T, q_start, h, out, *, miss_q, miss_phrase, miss_tier,
                              miss_count, policy=POLICY_LONGEST, gate=GATE_CONST, lam=1.0, sel_phrase=None,
                              sel_slot=None, flags=None, stream=None) -> None:
    """The lookup for callers that must not allocate: scratch is a fixed area of the library image,
    the miss list goes to caller-owned device buffers.  At most NOALLOC_MAX_ENTRIES (query, order)
    entries per call."""
    p = _params(policy, gate, lam)
    _check(lib().tfe_lookup_inject_noalloc(ctx, _addr(tokens), B, T, q_start, _addr(h), _addr(out), C.byref(p),
                                           _addr(sel_phrase), _addr(sel_slot), _addr(flags), _addr(miss_q),
                                           _addr(miss_phrase), _addr(miss_tier), _addr(miss_count),
                                           _stream(stream)), "tfe_lookup_inject_noalloc")


PREFETCH_MAX_BUDGET = 4096


def tfe_prefetch_candidates(ctx: int, history, B, H, cand_tokens, cand_prob, K, *, out_phrase, out_tier, out_score,
                            out_src, out_count, usefulness=None, benefit_host=1.0, benefit_ssd=2.0, budget=4096,
                            stream=None) -> None:
    p = TfePrefetchParams(float(benefit_host), float(benefit_ssd), int(budget))
    _check(lib().tfe_prefetch_candidates(ctx, _addr(history), B, H, _addr(cand_tokens), _addr(cand_prob), K,
                                         _addr(usefulness), C.byref(p), _addr(out_phrase), _addr(out_tier),
                                         _addr(out_score), _addr(out_src), _addr(out_count), _stream(stream)),
           "tfe_prefetch_candidates")


VICTIMS_MAX = 4096
INSTALL_DEVICE_MAX = 4096


def tfe_cache_install_device(ctx: int, n: int, phrase_ids, src_rows, dst_slots, applied=None, applied_count=None,
                             stream=None) -> None:
    """All arrays on the device; entries that cannot be applied are skipped."""
    _check(lib().tfe_cache_install_device(ctx, int(n), _addr(phrase_ids), _addr(src_rows), _addr(dst_slots),
                                          _addr(applied), _addr(applied_count), _stream(stream)),
           "tfe_cache_install_device")


def tfe_cache_policy_enable(ctx: int, stream=None) -> None:
    _check(lib().tfe_cache_policy_enable(ctx, _stream(stream)), "tfe_cache_policy_enable")


def tfe_cache_select_victims(ctx: int, n: int, half_life: int = 0, stream=None):
    """(slots int32[m], keys uint32[m]), m = min(n, gpu_slots), ascending (retention key, slot)."""
    slots, keys = np.empty(max(n, 1), np.int32), np.empty(max(n, 1), np.uint32)
    cnt = C.c_int32(0)
    _check(lib().tfe_cache_select_victims(ctx, int(n), int(half_life), _addr(slots), _addr(keys), C.byref(cnt),
                                          _stream(stream)), "tfe_cache_select_victims")
    return slots[:cnt.value], keys[:cnt.value]


def tfe_cache_select_tuning(ctx: int, list_cap: int = 0, final_cap: int = 0, n_samples: int = 0) -> None:
    _check(lib().tfe_cache_select_tuning(ctx, int(list_cap), int(final_cap), int(n_samples)), "tfe_cache_select_tuning")


def tfe_cache_select_victims_async(ctx: int, n: int, half_life: int = 0, stream=None) -> int:
    """Selection left on the device (see tfe_cache_select_victims_device); returns min(n, gpu_slots)."""
    cnt = C.c_int32(0)
    _check(lib().tfe_cache_select_victims(ctx, int(n), int(half_life), None, None, C.byref(cnt), _stream(stream)),
           "tfe_cache_select_victims")
    return cnt.value


def tfe_cache_select_victims_device(ctx: int):
    a, b = C.c_void_p(), C.c_void_p()
    _check(lib().tfe_cache_select_victims_device(ctx, C.byref(a), C.byref(b)), "tfe_cache_select_victims_device")
    return a.value, b.value


def tfe_cache_stats(ctx: int, gpu_slots: int, stream=None):
    """(freq uint32[C], last uint32[C], epoch)."""
    fl = np.empty((max(gpu_slots, 1), 2), np.uint32)
    ep = C.c_uint32(0)
    _check(lib().tfe_cache_stats(ctx, _addr(fl), C.byref(ep), _stream(stream)), "tfe_cache_stats")
    return fl[:gpu_slots, 0].copy(), fl[:gpu_slots, 1].copy(), ep.value


def tfe_miss_list(ctx: int, cap: int, stream=None, allow_overflow=False):
    """(q_idx uint32[n], phrase_id uint32[n], tier uint8[n], count) of the most recent lookup."""
    q = np.empty(max(cap, 1), np.uint32)
    ph = np.empty(max(cap, 1), np.uint32)
    tr = np.empty(max(cap, 1), np.uint8)
    cnt = C.c_int64(0)
    st = lib().tfe_miss_list(ctx, _addr(q), _addr(ph), _addr(tr), cap, C.byref(cnt), _stream(stream))
    if not (allow_overflow and st == TFE_ERR_MISS_OVERFLOW):
        _check(st, "tfe_miss_list")
    n = min(cnt.value, cap)
    return q[:n], ph[:n], tr[:n], cnt.value


def tfe_miss_list_device(ctx: int):
    """Device addresses (q_idx, phrase_id, tier, count) owned by the context."""
    a, b, c_, d = C.c_void_p(), C.c_void_p(), C.c_void_p(), C.c_void_p()
    _check(lib().tfe_miss_list_device(ctx, C.byref(a), C.byref(b), C.byref(c_), C.byref(d)),
           "tfe_miss_list_device")
    return a.value, b.value, c_.value, d.value


def tfe_destroy(ctx: int) -> None:
    if ctx:
        lib().tfe_destroy(ctx)


def tfe_index_geometry(ctx: int):
    a, b, c_ = C.c_int64(), C.c_int64(), C.c_int64()
    _check(lib().tfe_index_geometry(ctx, C.byref(a), C.byref(b), C.byref(c_)), "tfe_index_geometry")
    return a.value, b.value, c_.value


def tfe_launch_geometry(ctx: int):
    """(grid, block, queries per warp batch) of the most recent lookup."""
    g, b, t = C.c_int32(), C.c_int32(), C.c_int32()
    _check(lib().tfe_launch_geometry(ctx, C.byref(g), C.byref(b), C.byref(t)), "tfe_launch_geometry")
    return g.value, b.value, t.value


def tfe_set_tuning(ctx: int, batch_queries: int = 0) -> None:
    _check(lib().tfe_set_tuning(ctx, int(batch_queries)), "tfe_set_tuning")


def tfe_phrase_key64(vocab: int, tokens) -> tuple[int, bool]:
    t = np.ascontiguousarray(tokens, dtype=np.int32)
    ex = C.c_int32(0)
    k = lib().tfe_phrase_key64(vocab, _addr(t), len(t), C.byref(ex))
    return int(k), bool(ex.value)


def tfe_home_bucket(key: int, n_buckets: int) -> int:
    return int(lib().tfe_home_bucket(key, n_buckets))


# -- early-exit prefetch head -------------------------------------------------------------------
HEAD_MAX_K = 128
HEAD_MAX_BATCH = 256


def tfe_head_create(w_pref, V: int, d: int, max_batch: int) -> int:
    out = C.c_void_p()
    _check(lib().tfe_head_create(_addr(w_pref), int(V), int(d), int(max_batch), C.byref(out)), "tfe_head_create")
    return out.value


def tfe_head_destroy(head: int) -> None:
    lib().tfe_head_destroy(head)


def tfe_head_topk(head: int, hidden, B: int, K: int, cand_tokens, cand_prob, stream=None) -> None:
    _check(lib().tfe_head_topk(head, _addr(hidden), int(B), int(K), _addr(cand_tokens), _addr(cand_prob),
                               _stream(stream)), "tfe_head_topk")


def tfe_head_buffers(head: int):
    """Device addresses (logits fp32 [B][ld], ld, lse fp32 [B]) of the most recent call."""
    a, ld, b = C.c_void_p(), C.c_int64(0), C.c_void_p()
    _check(lib().tfe_head_buffers(head, C.byref(a), C.byref(ld), C.byref(b)), "tfe_head_buffers")
    return a.value, ld.value, b.value


def tfe_head_status(head: int, stream=None) -> int:
    """Synchronises; returns the device status word (0 = no wait ran out)."""
    flags = C.c_uint32(0)
    st = lib().tfe_head_status(head, C.byref(flags), _stream(stream))
    if st not in (TFE_OK, TFE_ERR_INTERNAL):
        _check(st, "tfe_head_status")
    return flags.value


def tfe_head_geometry(head: int):
    g, r, t = C.c_int32(0), C.c_int32(0), C.c_int32(0)
    _check(lib().tfe_head_geometry(head, C.byref(g), C.byref(r), C.byref(t)), "tfe_head_geometry")
    return g.value, r.value, t.value


MINE_HIST_BINS = 1024
MINE_MAX_TOKENS = 1 << 30


def tfe_mine_workspace_bytes(L: int, n_orders: int) -> int:
    return int(lib().tfe_mine_workspace_bytes(int(L), int(n_orders)))


def tfe_mine_ngrams(tokens, L: int, vocab: int, orders, min_count: int, cap: int, phrase_tokens=None, phrase_len=None,
                    phrase_count=None, want_hist: bool = True, workspace=None, workspace_bytes: int = 0, stream=None):
    """tokens and the three outputs on the device; returns (n_found, distinct int64 [n_orders], hist int64 [1024] or None)."""
    o = np.ascontiguousarray(orders, np.int32)
    found = C.c_int64(0)
    distinct = np.zeros(len(o), np.int64)
    hist = np.zeros(MINE_HIST_BINS, np.int64) if want_hist else None
    _check(lib().tfe_mine_ngrams(_addr(tokens), int(L), int(vocab), len(o), _addr(o), int(min_count), int(cap),
                                 _addr(phrase_tokens), _addr(phrase_len), _addr(phrase_count), C.byref(found),
                                 _addr(distinct), _addr(hist), _addr(workspace), int(workspace_bytes), _stream(stream)),
           "tfe_mine_ngrams")
    return found.value, distinct, hist


def tfe_assign_residency(count, N: int, gpu_slots: int, host_min_count: int, init_slot, stream=None):
    """count and init_slot on the device; returns (n_gpu, n_host, n_ssd)."""
    tiers = np.zeros(3, np.int64)
    _check(lib().tfe_assign_residency(_addr(count), int(N), int(gpu_slots), int(host_min_count), _addr(init_slot),
                                      _addr(tiers), _stream(stream)), "tfe_assign_residency")
    return tuple(int(x) for x in tiers)


def tfe_stream_copy(dst, src, nbytes: int, stream=None):
    """Streaming device copy of nbytes (a multiple of 16) bytes: the benchmark's same-footprint yardstick."""
    _check(lib().tfe_stream_copy(_addr(dst), _addr(src), int(nbytes), _stream(stream)), "tfe_stream_copy")
