"""GPU parity: the CUDA library against the CPU oracle, element by element, on
the same seeded inputs.  Integer outputs (phrase ids, slots, flags, miss lists)
must be bit-exact; hidden states within 2e-2 (bf16) / 1e-5 (fp32) of the exact
value.  Every call goes through the C ABI."""
import os

import numpy as np
import pytest
import torch

from paper_2607_07388_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def H():
    from paper_2607_07388_b200 import build
    build.build()
    from oracle import tfe_oracle
    tfe_oracle.build()
    import parity_harness
    return parity_harness


# ------------------------------------------------------------------ config 1


def test_config1_tiny_decode_all_modes(H):
    w = synth.config(1)
    tb, pr = H.pair_from_workload(w)
    tok = synth.make_queries(w, tb)
    h = synth.make_hidden_np(w)
    _, ref, info = pr.run_and_compare(tok, h, matcher="brute")
    assert 0.4 <= info["n_hit"] / w.Q <= 0.6, info          # ~50 % planted
    for lam in (0.0, 0.1, 0.5, 2.0):
        pr.run_and_compare(tok, h, lam=lam)
    pr.run_and_compare(tok, h, policy=1)
    pr.run_and_compare(tok, h, gate=1, lam=0.8)
    pr.run_and_compare(tok, h, policy=1, gate=1, lam=1.3)
    pr.run_and_compare(tok, h, in_place=True)
    pr.run_and_compare(tok, h, want_sel=False)
    pr.run_and_compare(tok, h[: w.B * (w.T - 5)], q_start=5)
    pr.close()


def test_repeat_runs_are_bitwise_identical(H):
    w = synth.config(1, residency="hot_host_ssd", gpu_slots=8000)
    tb, pr = H.pair_from_workload(w)
    tok = torch.from_numpy(synth.make_queries(w, tb)).to(H.DEV)
    h = pr.hidden_to_gpu(synth.make_hidden_np(w))
    a = pr.eng.lookup_inject(tok, h)
    la = pr.eng.miss_list()
    b = pr.eng.lookup_inject(tok, h)
    lb = pr.eng.miss_list()
    assert torch.equal(a.out.view(torch.int16), b.out.view(torch.int16))
    assert torch.equal(a.sel_phrase, b.sel_phrase) and torch.equal(a.flags, b.flags)
    assert la[3] == lb[3] > 0
    for x, y in zip(la[:3], lb[:3]):
        np.testing.assert_array_equal(x, y)
    pr.close()


# --------------------------------------------------- adversarial small tables


def _random_phrases(rng, alphabet, orders, count):
    phrases = set()
    total = sum(len(alphabet) ** n for n in orders)
    count = min(count, total // 2)
    while len(phrases) < count:
        n = int(rng.choice(orders))
        phrases.add(tuple(int(x) for x in rng.choice(alphabet, n)))
    return sorted(phrases, key=lambda p: rng.random())


@pytest.mark.parametrize("vocab,orders,load,hidden", [
    (6, (1, 2, 3, 4), 0.7, 0),              # every order packed
    (151_936, (2, 3, 4), 0.7, 0),           # order 4 hashed + verified
    (151_936, (2, 3, 4), 0.95, 0),          # crowded index: many cuckoo moves at build
    (1 << 20, (1, 3, 4), 0.9, 1),           # 20-bit ids, fp32 hidden states
    (70_000, (4,), 0.5, 0),
])
def test_small_tables_against_brute_force(H, vocab, orders, load, hidden):
    rng = np.random.default_rng(hash((vocab, orders)) % 1000)
    alphabet = np.array([0, 1, 2, 3, 4, vocab - 1])
    phrases = _random_phrases(rng, alphabet, orders, 700)
    pt, pl = H.phrases_to_arrays(phrases)
    N, C, d = len(phrases), len(phrases) + 5, 40
    state = rng.permutation(C)[:N].astype(np.int32)
    state[rng.random(N) < 0.2] = -1
    state[rng.random(N) < 0.1] = -2
    rows = synth.gaussian_bf16([1, vocab % 97], (C, d), 0.5)
    pr = H.Pair(pt, pl, state, rows, vocab=vocab, orders=orders, load_factor=load, hidden_dtype=hidden,
                max_kicks=100_000)
    B, T = 7, 53
    tok = rng.choice(np.concatenate([alphabet, [-1, vocab, 5]]), size=(B, T)).astype(np.int32)
    if hidden == 0:
        h = synth.gaussian_bf16([2], (B * T, d), 1.0)
    else:
        h = rng.standard_normal((B * T, d)).astype(np.float32)
    for policy in (0, 1):
        _, ref, info = pr.run_and_compare(tok, h, policy=policy, lam=0.75, matcher="brute")
        assert info["n_hit"] > 0 and info["n_miss"] > 0
    pr.run_and_compare(tok, h[:B * 3], q_start=50, policy=1, gate=1, lam=0.9, matcher="brute")
    pr.close()


def test_near_miss_queries_differ_in_one_token(H):
    # stored 4-grams vs queries that change exactly one token, and 2-/3-gram suffixes of stored 4-grams
    rng = np.random.default_rng(3)
    V = 151_936
    base = rng.integers(0, V, size=(400, 4)).astype(np.int32)
    phrases = [tuple(r) for r in base] + [tuple(r[1:]) for r in base[:100]] + [tuple(r[2:]) for r in base[50:150]]
    phrases = list(dict.fromkeys(phrases))
    pt, pl = H.phrases_to_arrays(phrases)
    N = len(phrases)
    rows = synth.gaussian_bf16([5], (N, 64), 0.1)
    pr = H.Pair(pt, pl, np.arange(N, dtype=np.int32), rows, vocab=V, orders=(2, 3, 4))
    q = np.repeat(base[:200], 5, axis=0)
    for k in range(4):
        q[k + 1::5, k] = (q[k + 1::5, k] + 1) % V          # row 0 intact, rows 1..4 one token off
    h = synth.gaussian_bf16([6], (len(q), 64), 1.0)
    _, ref, info = pr.run_and_compare(q, h, q_start=3, matcher="brute")
    assert (ref.flags[0::5] == 1).all()
    pr.close()


# ------------------------------------------------------------- shapes / edges


@pytest.mark.parametrize("d", [8, 24, 256, 1000, 2048, 4096])
@pytest.mark.parametrize("hidden", [0, 1])
def test_row_widths(H, d, hidden):
    w = synth.config(1, d=d, n_phrases=3000, gpu_slots=3000, B=3, T=29, p=0.5)
    tb = synth.make_table(w)
    pr = H.Pair(tb.phrase_tokens, tb.phrase_len, tb.init_slot, synth.make_rows_np(w, tb), vocab=w.vocab,
                orders=w.orders, hidden_dtype=hidden)
    tok = synth.make_queries(w, tb)
    h = synth.make_hidden_np(w)
    if hidden:
        h = synth.bf16_bits_to_f32(h) * np.float32(1.0009765625)
    pr.run_and_compare(tok, h, lam=0.5)
    pr.run_and_compare(tok, h, policy=1, gate=1, lam=0.5)
    pr.close()


def test_degenerate_calls(H):
    w = synth.config(1, n_phrases=500, gpu_slots=500, d=64)
    tb, pr = H.pair_from_workload(w)
    # one token, nothing can match (orders start at 2)
    pr.run_and_compare(np.array([[7]], np.int32), synth.make_hidden_np(w, Q=1))
    # Q = 0: q_start == T
    tok = torch.zeros((3, 4), dtype=torch.int32, device=H.DEV)
    e = torch.empty((0, 64), dtype=torch.bfloat16, device=H.DEV)
    pr.eng.lookup_inject(tok, e, q_start=4)
    assert pr.eng.miss_list()[3] == 0
    # all padding
    pad = np.full((2, 9), -1, np.int32)
    _, ref, info = pr.run_and_compare(pad, synth.make_hidden_np(w, Q=18))
    assert info["n_hit"] == 0 and info["n_miss"] == 0
    # a single sequence long enough to span several blocks with a ragged tail
    w2 = synth.config(1, n_phrases=500, gpu_slots=500, d=64, B=1, T=2051, p=0.3)
    tok2 = synth.make_queries(w2, tb)
    pr.run_and_compare(tok2, synth.make_hidden_np(w2))
    pr.close()


def test_empty_table(H):
    pt = np.zeros((0, 4), np.int32)
    pl = np.zeros(0, np.uint8)
    rows = np.zeros((4, 16), np.uint16)
    pr = H.Pair(pt, pl, np.zeros(0, np.int32), rows, vocab=100, orders=(2, 3))
    tok = np.arange(20, dtype=np.int32).reshape(2, 10)
    _, ref, info = pr.run_and_compare(tok, synth.gaussian_bf16([1], (20, 16), 1.0))
    assert info["n_hit"] == 0
    pr.close()


@pytest.mark.parametrize("load", [0.5, 0.7, 0.95])
def test_results_do_not_depend_on_load_factor(H, load):
    w = synth.config(1, load_factor=load, residency="hot_host_ssd", gpu_slots=9000)
    tb, pr = H.pair_from_workload(w, max_kicks=100_000)   # crowded tables need many moves at build
    tok = synth.make_queries(w, tb)
    pr.run_and_compare(tok, synth.make_hidden_np(w))
    pr.close()


def test_overfull_index_is_refused(H):
    from paper_2607_07388_b200 import binding as tfe
    w = synth.config(1, load_factor=1.0)        # every slot would have to be used: no cuckoo placement
    with pytest.raises(tfe.TfeError) as ei:
        H.pair_from_workload(w, max_kicks=50)
    assert ei.value.status == tfe.TFE_ERR_PROBE_LIMIT


# ------------------------------------------------ large calls, every batch size


@pytest.mark.parametrize("d,hidden,lam,orders", [
    (1024, 0, 1.0, (2, 3, 4)),      # packed bf16 fused multiply-add
    (1024, 0, 0.3, (2, 3)),         # fp32 arithmetic
    (1000, 0, 1.0, (2, 3, 4)),      # ragged vector tail
    (2048, 0, 0.5, (2, 3)),         # two chunks per row
    (2560, 1, 0.3, (2, 3, 4)),      # fp32 hidden states, five chunks per row
    (64, 0, 2.0, (2, 3)),           # short rows
    (512, 1, 0.7, (2, 3)),          # fp32 hidden states, one trip per row
])
def test_large_calls_all_batch_sizes(H, d, hidden, lam, orders):
    from paper_2607_07388_b200 import binding as tfe
    w = synth.config(3, n_phrases=30_000, gpu_slots=24_000, residency="hot_host_ssd", B=3, T=2731, d=d,
                     orders=orders, p=0.4, rows="procedural")
    tb = synth.make_table(w)
    pr = H.Pair(tb.phrase_tokens, tb.phrase_len, tb.init_slot, synth.make_rows_np(w, tb), vocab=w.vocab,
                orders=w.orders, hidden_dtype=hidden)
    tok = synth.make_queries(w, tb)
    h = synth.make_hidden_np(w)
    if hidden:
        h = synth.bf16_bits_to_f32(h) * np.float32(1.0009765625)
    seen = set()
    for qb in (0, 1, 3, 5, 8):          # 0: the library's own choice
        tfe.tfe_set_tuning(pr.eng.ctx, qb)
        _, ref, info = pr.run_and_compare(tok, h, lam=lam)
        seen.add(tfe.tfe_launch_geometry(pr.eng.ctx)[2])
        assert info["n_hit"] > 500 and info["n_miss"] > 50
        pr.run_and_compare(tok, h, lam=lam, in_place=True)
        pr.run_and_compare(tok, h[: w.B * (w.T - 2000)], lam=lam, q_start=2000, want_sel=False)
        pr.run_and_compare(tok, h, lam=lam, policy=1, gate=1)
        pr.run_and_compare(tok, h, lam=lam, gate=1)           # large and narrow enough for the gated LONGEST kernel
        pr.run_and_compare(tok, h, lam=lam, policy=1)
    cap = min(8, 32 // max(4, 2 * len(orders)))      # a query takes two lanes per order (at least four) of the warp
    assert {min(q, cap) for q in (1, 3, 5, 8)} <= seen
    pr.close()


# ------------------------------------------------------ miss list, cache install


def test_miss_list_overflow_and_device_view(H):
    from paper_2607_07388_b200 import binding as tfe
    w = synth.config(1, residency="hot_host_ssd", gpu_slots=6000, B=16, T=64)
    tb, pr = H.pair_from_workload(w)
    tok = synth.make_queries(w, tb)
    h = synth.make_hidden_np(w)
    _, ref, info = pr.run_and_compare(tok, h)
    n = info["n_miss"]
    assert n > 8
    q, ph, tr, cnt = pr.eng.miss_list(cap=5, allow_overflow=True)
    assert cnt == n and len(q) == 5
    np.testing.assert_array_equal(q, ref.miss_q[:5])
    with pytest.raises(tfe.TfeError) as ei:
        pr.eng.miss_list(cap=5)
    assert ei.value.status == tfe.TFE_ERR_MISS_OVERFLOW
    dq, dp, dt, dc = tfe.tfe_miss_list_device(pr.eng.ctx)
    torch.cuda.synchronize()

    class Raw:          # view context-owned device memory as a tensor
        def __init__(self, ptr, n, typestr):
            self.__cuda_array_interface__ = {"shape": (n,), "typestr": typestr, "data": (ptr, False), "version": 2}

    assert int(torch.as_tensor(Raw(dc, 1, "<i4"), device=H.DEV).cpu()[0]) == n
    np.testing.assert_array_equal(torch.as_tensor(Raw(dq, n, "<i4"), device=H.DEV).cpu().numpy().view(np.uint32),
                                  ref.miss_q)
    np.testing.assert_array_equal(torch.as_tensor(Raw(dp, n, "<i4"), device=H.DEV).cpu().numpy().view(np.uint32),
                                  ref.miss_phrase)
    np.testing.assert_array_equal(torch.as_tensor(Raw(dt, n, "|u1"), device=H.DEV).cpu().numpy(), ref.miss_tier)
    pr.close()


def test_cache_install_matches_the_oracle_state_machine(H):
    from paper_2607_07388_b200 import binding as tfe
    w = synth.config(1, residency="hot_host_ssd", n_phrases=6000, gpu_slots=4000, reserve_free=1500, B=16,
                     T=64, d=128, rows="procedural", p=0.45)
    tb, pr = H.pair_from_workload(w)
    tok = synth.make_queries(w, tb)
    h = synth.make_hidden_np(w)
    _, ref, info = pr.run_and_compare(tok, h)
    assert info["n_miss"] > 10
    ids = np.unique(ref.miss_phrase)
    half = ids[: len(ids) // 2]
    free = np.nonzero(pr.ora.slot_owner < 0)[0][: len(half)].astype(np.int32)
    src = synth.phrase_rows_np(w, half)
    # refusals leave both sides unchanged
    res0 = int(np.nonzero(tb.init_slot >= 0)[0][0])
    for bad_ids, bad_dst, status in (
            ([w.n_phrases], [0], tfe.TFE_ERR_UNKNOWN_PHRASE),
            ([res0], [int(free[0])], tfe.TFE_ERR_ALREADY_RESIDENT),
            ([int(half[0])], [w.gpu_slots], tfe.TFE_ERR_SLOT_RANGE),
            ([int(half[0]), int(half[0])], [int(free[0]), int(free[1])], tfe.TFE_ERR_INVALID_ARG),
            ([int(half[0]), int(half[1])], [int(free[0]), int(free[0])], tfe.TFE_ERR_INVALID_ARG)):
        with pytest.raises(tfe.TfeError) as ei:
            pr.eng.cache_install(bad_ids, src[: len(bad_ids)].copy(), bad_dst)
        assert ei.value.status == status
    pr.run_and_compare(tok, h)
    # install from pageable host memory into free slots
    pr.eng.cache_install(half, src, free)
    assert pr.ora.cache_install(half, src, free) == 0
    _, ref2, info2 = pr.run_and_compare(tok, h)
    assert info2["n_miss"] < info["n_miss"] and info2["n_hit"] > info["n_hit"]
    np.testing.assert_array_equal(H.bits_from_bf16_tensor(pr.rows_gpu), pr.ora.rows)
    # install the rest from device memory over OCCUPIED slots: their owners fall back to the host tier
    rest = np.unique(ref2.miss_phrase)
    victims = np.nonzero(pr.ora.slot_owner >= 0)[0][: len(rest)].astype(np.int32)
    src2 = synth.phrase_rows_np(w, rest)
    pr.eng.cache_install(rest, H.bf16_tensor_from_bits(src2, H.DEV), victims)
    assert pr.ora.cache_install(rest, src2, victims) == 0
    pr.run_and_compare(tok, h)
    np.testing.assert_array_equal(H.bits_from_bf16_tensor(pr.rows_gpu), pr.ora.rows)
    # pinned host source
    more = np.nonzero(pr.ora.slot_state < 0)[0][:64].astype(np.uint32)
    dst = np.nonzero(pr.ora.slot_owner < 0)[0][:64].astype(np.int32)
    src3 = synth.phrase_rows_np(w, more)
    pinned = torch.from_numpy(src3.view(np.int16)).pin_memory()
    pr.eng.cache_install(more, pinned, dst)
    assert pr.ora.cache_install(more, src3, dst) == 0
    pr.run_and_compare(tok, h, policy=1)
    pr.close()


def test_host_buffer_entry_point(H):
    from paper_2607_07388_b200 import binding as tfe
    w = synth.config(1, residency="hot_host", gpu_slots=12000)
    tb, pr = H.pair_from_workload(w)
    tok = synth.make_queries(w, tb)
    h = synth.make_hidden_np(w)
    out = np.empty_like(h)
    sp = np.empty(w.Q, np.uint32); ss = np.empty(w.Q, np.int32); fl = np.empty(w.Q, np.uint8)
    tfe.tfe_lookup_inject_host(pr.eng.ctx, tok, w.B, w.T, 0, h, out, lam=1.0, sel_phrase=sp, sel_slot=ss,
                               flags=fl)
    mq, mp, mt, cnt = pr.eng.miss_list()
    ref = pr.ora.lookup(tok)
    _, rounded = pr.ora.inject(ref, h, lam=1.0)
    np.testing.assert_array_equal(sp, ref.sel_phrase)
    np.testing.assert_array_equal(ss, ref.sel_slot)
    np.testing.assert_array_equal(fl, ref.flags)
    np.testing.assert_array_equal(out, rounded)
    np.testing.assert_array_equal(mq, ref.miss_q)
    pr.close()


def test_host_buffer_entry_point_in_pieces(H):
    """A host-buffer call large enough to be issued as several launches over query ranges
    (copies and kernels overlapped): every output and the ordered miss list of the whole call
    must equal the oracle's, call after call, and a plain device call afterwards must be
    unaffected.  T is odd so the pieces end inside sequences."""
    from paper_2607_07388_b200 import binding as tfe
    w = synth.config(1, B=6, T=2731, d=1024, n_phrases=60_000, gpu_slots=40_000, residency="hot_host", p=0.6)
    assert w.Q * w.d * 2 >= 32 << 20
    tb, pr = H.pair_from_workload(w)
    h = synth.make_hidden_np(w)
    for variant in (0, 1):
        tok = synth.make_queries(w, tb, variant=variant)
        out = np.empty_like(h)
        sp = np.empty(w.Q, np.uint32); ss = np.empty(w.Q, np.int32); fl = np.empty(w.Q, np.uint8)
        tfe.tfe_lookup_inject_host(pr.eng.ctx, tok, w.B, w.T, 0, h, out, lam=1.0, sel_phrase=sp, sel_slot=ss,
                                   flags=fl)
        mq, mp, mt, cnt = pr.eng.miss_list()
        ref = pr.ora.lookup(tok)
        _, rounded = pr.ora.inject(ref, h, lam=1.0)
        np.testing.assert_array_equal(sp, ref.sel_phrase)
        np.testing.assert_array_equal(ss, ref.sel_slot)
        np.testing.assert_array_equal(fl, ref.flags)
        np.testing.assert_array_equal(out, rounded)
        assert cnt == len(ref.miss_q) and cnt > 1000
        assert len(np.unique(ref.miss_q // 2048)) > 4        # misses in many pieces
        np.testing.assert_array_equal(mq, ref.miss_q)
        np.testing.assert_array_equal(mp, ref.miss_phrase)
        np.testing.assert_array_equal(mt, ref.miss_tier)
    pr.run_and_compare(tok, h, lam=1.0)
    pr.close()


@pytest.mark.parametrize("seed", range(min(30, int(os.environ.get("TFE_RANDOM_CASES", "4")))))
def test_host_buffer_pieces_random_shapes(H, seed):
    """Host-buffer calls large enough to go in pieces, with seeded random shapes: piece boundaries
    fall anywhere in the sequences, pieces may hold no hit or no miss at all."""
    from paper_2607_07388_b200 import binding as tfe
    rng = np.random.default_rng([909, seed])
    d = int(rng.choice([512, 1024, 2048, 4104]))
    Q_target = int(rng.integers(16 << 20, 72 << 20)) // (2 * d) + 1
    shape = "prefill" if rng.random() < 0.6 else "decode"
    orders = (2, 3) if rng.random() < 0.5 else (2, 3, 4)
    if shape == "prefill":
        B = int(rng.integers(1, 9)); T = Q_target // B + 1
    else:
        B = Q_target; T = max(orders)
    w = synth.config(1, shape=shape, B=B, T=T, d=d, orders=orders, n_phrases=40_000, gpu_slots=15_000,
                     residency=str(rng.choice(["hot_host", "hot_host_ssd"])), p=float(rng.uniform(0.05, 0.5)))
    assert w.Q * w.d * 2 >= 16 << 20
    tb, pr = H.pair_from_workload(w)
    tok = synth.make_queries(w, tb)
    h = synth.make_hidden_np(w)
    out = np.empty_like(h)
    sp = np.empty(w.Q, np.uint32); ss = np.empty(w.Q, np.int32); fl = np.empty(w.Q, np.uint8)
    lam = float(rng.choice([1.0, 0.5, 0.3]))
    tfe.tfe_lookup_inject_host(pr.eng.ctx, tok, w.B, w.T, w.q_start, h, out, lam=lam, sel_phrase=sp, sel_slot=ss, flags=fl)
    mq, mp, mt, cnt = pr.eng.miss_list()
    ref = pr.ora.lookup(tok, w.q_start)
    np.testing.assert_array_equal(sp, ref.sel_phrase)
    np.testing.assert_array_equal(ss, ref.sel_slot)
    np.testing.assert_array_equal(fl, ref.flags)
    assert cnt == len(ref.miss_q)
    np.testing.assert_array_equal(mq, ref.miss_q)
    np.testing.assert_array_equal(mp, ref.miss_phrase)
    np.testing.assert_array_equal(mt, ref.miss_tier)
    exact, rounded = pr.ora.inject(ref, h, lam=lam)
    if lam != 0.3:
        np.testing.assert_array_equal(out, rounded)
    else:
        assert np.abs(synth.bf16_bits_to_f32(out).astype(np.float64) - exact).max() <= 2e-2
    pr.close()
