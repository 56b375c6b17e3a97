"""CPU-side checks of the C-ABI library: it loads, exports what the header
declares, refuses bad arguments before touching a device, and its key / bucket
functions are exact and uniform.  No kernel is launched here."""
import ctypes as C
import os
import re

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def tfe():
    from paper_2607_07388_b200 import binding, build
    build.build()
    binding.lib()
    return binding


def test_library_exports_every_declared_symbol(tfe):
    header = open(os.path.join(ROOT, "include", "tfe.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(tfe_[a-z0-9_]+)\s*\(", header))
    assert declared == set(tfe.EXPORTS)
    L = tfe.lib()
    for name in declared:
        assert getattr(L, name) is not None


def test_status_strings(tfe):
    seen = {tfe.lib().tfe_status_string(i).decode() for i in range(12)}
    assert len(seen) == 12 and "ok" in seen


def _build_status(tfe, cfg, pt, pl, sl, rows_addr=0x1000):
    out = C.c_void_p()
    return tfe.lib().tfe_index_build(C.byref(cfg), pt.ctypes.data, pl.ctypes.data, sl.ctypes.data,
                                     rows_addr, None, C.byref(out))


def test_build_refuses_bad_arguments_on_the_host(tfe):
    pt = np.array([[1, 2, -1, -1], [3, 4, 5, -1]], np.int32)
    pl = np.array([2, 3], np.uint8)
    sl = np.array([0, -1], np.int32)
    ok = dict(d=16, vocab=10, orders=(2, 3), n_phrases=2, gpu_slots=2)
    bad_cfgs = [dict(ok, d=12), dict(ok, d=0), dict(ok, vocab=0), dict(ok, orders=(3, 2)),
                dict(ok, orders=(0, 2)), dict(ok, orders=(2, 5)), dict(ok, load_factor=0.0),
                dict(ok, load_factor=1.5), dict(ok, hidden_dtype=2), dict(ok, gpu_slots=-1)]
    for kw in bad_cfgs:
        assert _build_status(tfe, tfe.make_config(**kw), pt, pl, sl) == tfe.TFE_ERR_INVALID_ARG, kw
    cfg = tfe.make_config(**ok)
    assert _build_status(tfe, cfg, pt, pl, sl, rows_addr=0x1004) == tfe.TFE_ERR_INVALID_ARG   # misaligned rows
    assert _build_status(tfe, cfg, pt, np.array([2, 4], np.uint8), sl) == tfe.TFE_ERR_INVALID_ARG  # 4 not an order
    bad_tok = pt.copy(); bad_tok[1, 2] = 10
    assert _build_status(tfe, cfg, bad_tok, pl, sl) == tfe.TFE_ERR_INVALID_ARG
    assert _build_status(tfe, cfg, pt, pl, np.array([0, 2], np.int32)) == tfe.TFE_ERR_SLOT_RANGE
    assert _build_status(tfe, cfg, pt, pl, np.array([1, 1], np.int32)) == tfe.TFE_ERR_SLOT_RANGE
    assert _build_status(tfe, cfg, pt, pl, np.array([0, -3], np.int32)) == tfe.TFE_ERR_INVALID_ARG
    dup = np.array([[1, 2, -1, -1], [1, 2, -1, -1]], np.int32)
    assert _build_status(tfe, tfe.make_config(**dict(ok, orders=(2,))), dup, np.array([2, 2], np.uint8), sl) \
        == tfe.TFE_ERR_DUPLICATE_PHRASE


def test_packed_keys_are_injective_and_nonzero(tfe):
    # every tuple of orders 1..3 over a small vocabulary: all keys distinct, none zero
    V = 13
    keys = {}
    for n in (1, 2, 3):
        for idx in np.ndindex(*([V] * n)):
            k, exact = tfe.tfe_phrase_key64(V, idx)
            assert exact and k != 0
            assert k not in keys, (idx, keys.get(k))
            keys[k] = idx
    # the benchmark vocabulary: orders <= 3 are packed (3 * 18 bits), order 4 is hashed + verified
    V = 151_936
    assert tfe.tfe_phrase_key64(V, [V - 1, 0, V - 1])[1] is True
    assert tfe.tfe_phrase_key64(V, [1, 2, 3, 4])[1] is False
    # token order matters, padding gives no key
    assert tfe.tfe_phrase_key64(V, [1, 2])[0] != tfe.tfe_phrase_key64(V, [2, 1])[0]
    assert tfe.tfe_phrase_key64(V, [1, 2, 3, 4])[0] != tfe.tfe_phrase_key64(V, [4, 3, 2, 1])[0]
    assert tfe.tfe_phrase_key64(V, [1, V])[0] == 0 and tfe.tfe_phrase_key64(V, [-1, 2])[0] == 0
    # extreme corners stay distinct
    corner = {tfe.tfe_phrase_key64(V, t)[0] for t in ([0, 0], [0, 0, 0], [0, 1], [1, 0], [0, 0, 1], [V - 1, V - 1],
                                                        [V - 1, V - 1, V - 1], [0], [V - 1])}
    assert len(corner) == 9


def test_home_buckets_follow_the_papers_occupancy_formula(tfe):
    # M phrase keys into B buckets: the number of distinct home buckets must match the closed form
    # B * (1 - (1 - 1/B)^M) the paper gives for uniform hashing (Sec. 3.1), within 1 %.
    rng = np.random.default_rng(7)
    V = 151_936
    for M, B, n in ((200_000, 200_000, 2), (200_000, 50_000, 3), (100_000, 142_858, 4), (50_000, 7_919, 2)):
        toks = rng.integers(0, V, size=(M, n)).astype(np.int32)
        toks[: M // 2, 0] = toks[0, 0]            # half the phrases share their first token
        toks = np.unique(toks, axis=0)
        homes = {tfe.tfe_home_bucket(tfe.tfe_phrase_key64(V, t)[0], B) for t in toks}
        assert max(homes) < B
        expect = B * (1.0 - (1.0 - 1.0 / B) ** len(toks))
        assert abs(len(homes) - expect) / expect < 0.01, (M, B, n, len(homes), expect)


def test_index_bytes_per_entry_below_the_papers_overhead():
    # The paper's 100M-entry table takes 215.86 GB with 1024-dim FP16 vectors (Sec. 5.3):
    # 2158.6 B per entry, of which 2048 B are the vector, so ~110 B of index + metadata.
    paper_overhead = 215.86e9 / 100e6 - 2048
    assert 100 < paper_overhead < 120
    ours = 16 / 0.7 + 4 + 4 + 16        # index slot / load factor + position + owner + stored tuple
    assert ours < paper_overhead


def test_header_is_plain_c(tmp_path):
    """The boundary is a C ABI: the header must compile as C11 with nothing but the standard headers,
    and a C program must link against the library by name."""
    import subprocess
    src = tmp_path / "use_tfe.c"
    src.write_text('#include "tfe.h"\n'
                   'int main(void) {\n'
                   '    tfe_config cfg; tfe_inject_params prm; tfe_prefetch_params pf;\n'
                   '    (void)cfg; (void)prm; (void)pf;\n'
                   '    return tfe_status_string(TFE_OK) == 0;\n'
                   '}\n')
    inc = os.path.join(ROOT, "include")
    subprocess.run(["gcc", "-std=c11", "-Wall", "-Werror", "-pedantic", "-fsyntax-only", f"-I{inc}", str(src)], check=True)
    from paper_2607_07388_b200 import build
    lib = build.build()
    exe = tmp_path / "use_tfe"
    subprocess.run(["gcc", "-std=c11", f"-I{inc}", str(src), lib, "-o", str(exe),
                    f"-Wl,-rpath,{os.path.dirname(lib)}"], check=True)
    assert subprocess.run([str(exe)]).returncode == 0


def test_new_entry_points_refuse_bad_arguments_on_the_host(tfe):
    """Argument errors come back before any device call (this box has no GPU)."""
    L = tfe.lib()
    out = C.c_void_p()
    # early-exit head
    for w, V, d, mb in ((None, 100, 64, 4), (0x1000, 0, 64, 4), (0x1000, 100, 32, 4), (0x1000, 100, 96, 4),
                        (0x1000, 100, 64, 0), (0x1000, 100, 64, 257), (0x1004, 100, 64, 4)):
        assert L.tfe_head_create(w, V, d, mb, C.byref(out)) == tfe.TFE_ERR_INVALID_ARG, (w, V, d, mb)
        assert out.value is None
    assert L.tfe_head_create(0x1000, 100, 64, 4, None) == tfe.TFE_ERR_INVALID_ARG
    assert L.tfe_head_topk(None, 0x1000, 1, 1, 0x1000, 0x1000, None) == tfe.TFE_ERR_INVALID_ARG
    flags = C.c_uint32(0)
    assert L.tfe_head_status(None, C.byref(flags), None) == tfe.TFE_ERR_INVALID_ARG
    assert L.tfe_head_geometry(None, None, None, None) == tfe.TFE_ERR_INVALID_ARG
    L.tfe_head_destroy(None)                                    # a no-op
    # retention ranking
    cnt = C.c_int32(0)
    assert L.tfe_cache_policy_enable(None, None) == tfe.TFE_ERR_INVALID_ARG
    assert L.tfe_cache_select_victims(None, 4, 0, 0x1000, None, C.byref(cnt), None) == tfe.TFE_ERR_INVALID_ARG
    assert L.tfe_cache_stats(None, None, None, None) == tfe.TFE_ERR_INVALID_ARG
    # device build: the same configuration checks as the host build
    pt = np.zeros((2, 4), np.int32)
    for kw in (dict(d=12), dict(orders=(3, 2)), dict(load_factor=0.0), dict(hidden_dtype=2)):
        cfg = tfe.make_config(**dict(dict(d=16, vocab=10, orders=(2, 3), n_phrases=2, gpu_slots=2), **kw))
        assert L.tfe_index_build_device(C.byref(cfg), pt.ctypes.data, 0x1000, 0x1000, 0x1000, None, C.byref(out)) \
            == tfe.TFE_ERR_INVALID_ARG, kw
    cfg = tfe.make_config(d=16, vocab=10, orders=(2, 3), n_phrases=2, gpu_slots=2)
    assert L.tfe_index_build_device(C.byref(cfg), None, 0x1000, 0x1000, 0x1000, None, C.byref(out)) == tfe.TFE_ERR_INVALID_ARG
    assert L.tfe_index_build_device(C.byref(cfg), 0x1004, 0x1000, 0x1000, 0x1000, None, C.byref(out)) == tfe.TFE_ERR_INVALID_ARG
    # device-side installation
    assert L.tfe_cache_install_device(None, 4, 0x1000, 0x1000, 0x1000, None, None, None) == tfe.TFE_ERR_INVALID_ARG
    # n-gram extraction: every refusal below happens before the first device call
    found = C.c_int64(7)
    orders = np.array([2, 3], np.int32)
    bad = np.array([3, 2], np.int32)
    mine = lambda tok, Ln, vocab, n_o, o, cap, pt_, ws, wsb: L.tfe_mine_ngrams(
        tok, Ln, vocab, n_o, o, 1, cap, pt_, 0x1000, 0x1000, C.byref(found), None, None, ws, wsb, None)
    assert mine(0x1000, -1, 10, 2, orders.ctypes.data, 0, None, None, 0) == tfe.TFE_ERR_INVALID_ARG
    assert mine(0x1000, (1 << 30) + 1, 10, 2, orders.ctypes.data, 0, None, None, 0) == tfe.TFE_ERR_INVALID_ARG
    assert mine(0x1000, 16, 0, 2, orders.ctypes.data, 0, None, None, 0) == tfe.TFE_ERR_INVALID_ARG
    assert mine(0x1000, 16, 10, 2, bad.ctypes.data, 0, None, None, 0) == tfe.TFE_ERR_INVALID_ARG
    assert mine(0x1000, 16, 10, 5, orders.ctypes.data, 0, None, None, 0) == tfe.TFE_ERR_INVALID_ARG
    assert mine(None, 16, 10, 2, orders.ctypes.data, 0, None, None, 0) == tfe.TFE_ERR_INVALID_ARG
    assert mine(0x1000, 16, 10, 2, orders.ctypes.data, 4, None, None, 0) == tfe.TFE_ERR_INVALID_ARG         # cap without outputs
    assert mine(0x1000, 16, 10, 2, orders.ctypes.data, 4, 0x1004, None, 0) == tfe.TFE_ERR_INVALID_ARG       # misaligned tuples
    assert mine(0x1000, 16, 10, 2, orders.ctypes.data, 0, None, None, 64) == tfe.TFE_ERR_INVALID_ARG        # size without buffer
    assert mine(0x1000, 16, 10, 2, orders.ctypes.data, 0, None, 0x1000, 64) == tfe.TFE_ERR_CAPACITY         # workspace too small
    assert mine(None, 0, 10, 2, orders.ctypes.data, 0, None, None, 0) == tfe.TFE_OK and found.value == 0   # empty corpus: no device call
    assert L.tfe_mine_workspace_bytes(-1, 2) == -1 and L.tfe_mine_workspace_bytes(16, 0) == -1
    assert L.tfe_mine_workspace_bytes(1 << 20, 3) >= (1 << 21) * 16 + 4 * 4 * (1 << 20)     # table + one array per order + bigram slots
    # initial residency: refusals before any device call; N = 0 touches nothing
    tiers = np.zeros(3, np.int64)
    assert L.tfe_assign_residency(0x1000, -1, 4, 2, 0x1000, tiers.ctypes.data, None) == tfe.TFE_ERR_INVALID_ARG
    assert L.tfe_assign_residency(0x1000, 1 << 31, 4, 2, 0x1000, tiers.ctypes.data, None) == tfe.TFE_ERR_INVALID_ARG
    assert L.tfe_assign_residency(0x1000, 8, -1, 2, 0x1000, tiers.ctypes.data, None) == tfe.TFE_ERR_INVALID_ARG
    assert L.tfe_assign_residency(None, 8, 4, 2, 0x1000, tiers.ctypes.data, None) == tfe.TFE_ERR_INVALID_ARG
    assert L.tfe_assign_residency(0x1000, 8, 4, 2, None, tiers.ctypes.data, None) == tfe.TFE_ERR_INVALID_ARG
    assert L.tfe_assign_residency(None, 0, 4, 2, None, tiers.ctypes.data, None) == tfe.TFE_OK and tiers.tolist() == [0, 0, 0]
