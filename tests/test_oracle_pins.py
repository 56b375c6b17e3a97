"""Pins for the CPU oracle: every expected value here comes from the paper's
definitions worked by hand, a closed form, a library routine, or an independent
brute-force written in this file -- never from the oracle itself."""
import os

import numpy as np
import pytest
import torch

from paper_2607_07388_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def bf(x):
    """float(s) -> bf16 bit patterns via torch's float32->bfloat16 conversion (library routine)."""
    t = torch.tensor(np.asarray(x, dtype=np.float32)).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16).copy()


def unbf(b):
    t = torch.from_numpy(np.asarray(b, dtype=np.uint16).view(np.int16).copy()).view(torch.bfloat16)
    return t.to(torch.float64).numpy()


def mk_oracle(orc, phrases, slots, rows, d, vocab, orders, C):
    pt = np.full((len(phrases), 4), -1, np.int32)
    pl = np.zeros(len(phrases), np.uint8)
    for i, p in enumerate(phrases):
        pt[i, :len(p)] = p
        pl[i] = len(p)
    return orc.Oracle(pt, pl, np.asarray(slots, np.int32), rows, d=d, vocab=vocab, orders=orders,
                      gpu_slots=C)


# ---------------------------------------------------------------- bf16 codec


def test_bf16_decode_matches_library(oracle_mod):
    bits = np.concatenate([np.arange(0, 0x7F80, 37, dtype=np.uint16),
                           np.arange(0x8000, 0xFF80, 41, dtype=np.uint16),
                           np.array([0, 1, 0x007F, 0x0080, 0x7F7F, 0x8000, 0x3F80], np.uint16)])
    np.testing.assert_array_equal(oracle_mod.bf16_to_double(bits), unbf(bits))


def test_bf16_encode_matches_library_on_float32_inputs(oracle_mod):
    rng = np.random.default_rng(0)
    x = np.concatenate([rng.standard_normal(4000).astype(np.float32) * 3,
                        (rng.standard_normal(500) * 1e-3).astype(np.float32),
                        np.array([0.0, -0.0, 1.0, -1.0, 1e38, -1e38, 1e-40, 3.3895e38], np.float32)])
    # exact ties between two bf16 neighbours: odd and even significands
    ties = np.array([1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, -(2.0 + 2.0 ** -7), 0.75 + 2.0 ** -9], np.float32)
    x = np.concatenate([x, ties])
    np.testing.assert_array_equal(oracle_mod.bf16_from_double(x.astype(np.float64)), bf(x))


def test_bf16_encode_rounds_the_real_number_not_its_float32(oracle_mod):
    # 1 + 2^-8 is a tie (-> 1.0, even); a hair above it must go up, a hair below it down,
    # even though float32 cannot tell them from the tie.
    up = oracle_mod.bf16_from_double(np.array([1.0 + 2.0 ** -8 + 2.0 ** -40]))
    dn = oracle_mod.bf16_from_double(np.array([1.0 + 2.0 ** -8 - 2.0 ** -40]))
    assert unbf(up)[0] == 1.0 + 2.0 ** -7
    assert unbf(dn)[0] == 1.0
    # overflow, subnormals, signed zero
    assert oracle_mod.bf16_from_double(np.array([1e39]))[0] == 0x7F80
    assert oracle_mod.bf16_from_double(np.array([-1e39]))[0] == 0xFF80
    assert oracle_mod.bf16_from_double(np.array([2.0 ** -133]))[0] == 0x0001
    assert oracle_mod.bf16_from_double(np.array([2.0 ** -135]))[0] == 0x0000
    assert oracle_mod.bf16_from_double(np.array([-0.0]))[0] == 0x8000


# ------------------------------------------------- exact match and selection


def _load_worked():
    rows = []
    with open(os.path.join(GOLDEN, "worked_lookup.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            rows.append([int(v) for v in line.split()])
    return np.array(rows)


WORKED_PHRASES = [(11, 12), (10, 11, 12), (12, 13), (13, 14), (12, 13, 14), (14, 14)]
WORKED_SLOTS = [3, 0, -1, -2, 2, 1]
WORKED_STREAM = [[10, 11, 12, 13, 14, 14, 99, 14, 14]]


@pytest.mark.parametrize("matcher", ["brute", "sorted"])
def test_worked_lookup_longest_and_all(oracle_mod, matcher):
    g = _load_worked()
    o = mk_oracle(oracle_mod, WORKED_PHRASES, WORKED_SLOTS, np.zeros((4, 8), np.uint16), 8, 100,
                  [2, 3], 4)
    tok = np.array(WORKED_STREAM, np.int32)
    r = o.lookup(tok, 0, oracle_mod.POLICY_LONGEST, matcher)
    np.testing.assert_array_equal(r.match, g[:, 1:3])
    np.testing.assert_array_equal(r.sel_phrase.astype(np.int64),
                                  np.where(g[:, 3] < 0, 0xFFFFFFFF, g[:, 3]))
    np.testing.assert_array_equal(r.sel_slot, g[:, 4])
    np.testing.assert_array_equal(r.flags, g[:, 5])
    assert list(zip(r.miss_q, r.miss_phrase, r.miss_tier)) == [(3, 2, 2)]
    ra = o.lookup(tok, 0, oracle_mod.POLICY_ALL, matcher)
    assert list(zip(ra.miss_q, ra.miss_phrase, ra.miss_tier)) == [(3, 2, 2), (4, 3, 3)]
    assert ra.flags.tolist()[4] == [3, 1] and ra.sel_slot.tolist()[4] == [-2, 2]
    assert ra.flags.tolist()[2] == [1, 1] and ra.sel_phrase.tolist()[2] == [0, 1]


def test_q_start_sequence_start_and_padding(oracle_mod):
    # two sequences; an n-gram never crosses the start of its own sequence, ids outside
    # [0, vocab) break every n-gram that contains them; ids 0 and vocab-1 are ordinary tokens.
    V = 50
    phrases = [(0, 49), (49, 0, 49), (7, 7), (7, 7, 7), (49, 7)]
    o = mk_oracle(oracle_mod, phrases, [0, 1, 2, 3, 4], np.zeros((5, 8), np.uint16), 8, V, [2, 3], 5)
    tok = np.array([[49, 0, 49, 7, 7, 7, 7],
                    [7, 7, -1, 7, 7, 50, 49]], np.int32)
    r = o.lookup(tok, 0)
    # seq 0: t0 none | t1 (49,0) none | t2 (0,49)->0,(49,0,49)->1 | t3 (49,7)->4 | t4 (7,7)->2 |
    #        t5 (7,7)->2,(7,7,7)->3 | t6 same
    # seq 1: t0 none (the 49 7 of the previous row must not leak) | t1 (7,7)->2 | t2 pad | t3 pad in gram |
    #        t4 (7,7)->2 ; 3-gram holds the pad | t5 pad(50) | t6 pad in gram
    exp = [-1, -1, 1, 4, 2, 3, 3, -1, 2, -1, -1, 2, -1, -1]
    np.testing.assert_array_equal(r.sel_phrase.astype(np.int64), np.where(np.array(exp) < 0, 0xFFFFFFFF, exp))
    # q_start = 4 keeps only t in [4, 7) of each sequence, numbered b*3 + (t-4)
    r2 = o.lookup(tok, 4)
    np.testing.assert_array_equal(r2.sel_phrase.astype(np.int64),
                                  np.where(np.array(exp[4:7] + exp[11:14]) < 0, 0xFFFFFFFF,
                                           exp[4:7] + exp[11:14]))


def _dict_matcher(phrases, tok, q_start, vocab, orders):
    """Independent matcher: python dict keyed by the token tuple."""
    table = {tuple(int(x) for x in p): i for i, p in enumerate(phrases)}
    B, T = tok.shape
    out = []
    for b in range(B):
        for t in range(q_start, T):
            row = []
            for n in orders:
                g = tuple(int(x) for x in tok[b, t - n + 1:t + 1]) if t - n + 1 >= 0 else ()
                ok = len(g) == n and all(0 <= x < vocab for x in g)
                row.append(table.get(g, -1) if ok else -1)
            out.append(row)
    return np.array(out, np.int64)


@pytest.mark.parametrize("seed,orders", [(1, [2, 3]), (2, [1, 2, 3, 4]), (3, [2, 4]), (4, [3])])
def test_matchers_agree_with_dict_brute_force(oracle_mod, seed, orders):
    # tiny alphabet so that phrases share prefixes/suffixes, nest inside each other and
    # differ from stream n-grams in exactly one token all the time
    rng = np.random.default_rng(seed)
    V = 6
    phrases = set()
    target = min(300, sum(V ** n for n in orders) // 2)
    while len(phrases) < target:
        n = int(rng.choice(orders))
        phrases.add(tuple(int(x) for x in rng.integers(0, V, n)))
    phrases = sorted(phrases, key=lambda p: rng.random())
    slots = rng.permutation(len(phrases)).astype(np.int32)
    o = mk_oracle(oracle_mod, phrases, slots, np.zeros((len(phrases), 8), np.uint16), 8, V, orders,
                  len(phrases))
    tok = rng.integers(-1, V + 1, size=(5, 40)).astype(np.int32)
    for q_start in (0, 3, 39):
        exp = _dict_matcher(phrases, tok, q_start, V, orders)
        np.testing.assert_array_equal(o.match(tok, q_start, "brute"), exp)
        np.testing.assert_array_equal(o.match(tok, q_start, "sorted"), exp)


def test_duplicate_tuple_is_refused(oracle_mod):
    o = mk_oracle(oracle_mod, [(1, 2), (3, 4, 5), (1, 2)], [0, 1, 2], np.zeros((3, 8), np.uint16), 8,
                  10, [2, 3], 3)
    with pytest.raises(ValueError):
        o.sorted_perm()


# ----------------------------------------------------------------- injection


def _one_hit_oracle(oracle_mod, row_vals, d=8, slot=1, C=3, state=None):
    rows = np.zeros((C, d), np.uint16)
    rows[slot] = bf(row_vals)
    o = mk_oracle(oracle_mod, [(1, 2)], [slot if state is None else state], rows, d, 10, [2], C)
    tok = np.array([[1, 2, 3]], np.int32)      # q0 absent (no 2-gram), q1 hit, q2 absent
    return o, tok


def test_injection_equation_by_hand(oracle_mod):
    d = 8
    row = [0.5, -0.25, 2.0, 0.0, 1.0, 2.0 ** -8, 3 * 2.0 ** -8, -1.5]
    o, tok = _one_hit_oracle(oracle_mod, row)
    hval = np.array([[9, 9, 9, 9, 9, 9, 9, 9],
                     [1.0, 1.0, -4.0, 0.75, -1.0, 1.0, 1.0, 0.5],
                     [7, 7, 7, 7, 7, 7, 7, 7]], np.float32)
    h = bf(hval)
    r = o.lookup(tok)
    assert r.flags.tolist() == [0, 1, 0]
    exact, rounded = o.inject(r, h, lam=1.0)
    # h + 1.0 * row, real numbers
    np.testing.assert_array_equal(exact[1], [1.5, 0.75, -2.0, 0.75, 0.0, 1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, -1.0])
    # bf16: 1+2^-8 is a tie -> even (1.0); 1+3*2^-8 is a tie -> even (1+2^-6)
    np.testing.assert_array_equal(unbf(rounded[1]), [1.5, 0.75, -2.0, 0.75, 0.0, 1.0, 1.0 + 2.0 ** -6, -1.0])
    # rows 0 and 2: absent -> bitwise h
    np.testing.assert_array_equal(rounded[[0, 2]], h[[0, 2]])
    np.testing.assert_array_equal(exact[[0, 2]], hval[[0, 2]].astype(np.float64))
    # lambda = 0.25
    exact, rounded = o.inject(r, h, lam=0.25)
    np.testing.assert_array_equal(exact[1, :5], [1.125, 0.9375, -3.5, 0.75, -0.75])


def test_injection_closed_forms(oracle_mod):
    rng = np.random.default_rng(5)
    d = 64
    m = rng.standard_normal(d).astype(np.float32)
    o, tok = _one_hit_oracle(oracle_mod, m, d=d)
    r = o.lookup(tok)
    h = bf(rng.standard_normal((3, d)))
    # lambda = 0: identity, bitwise
    _, out = o.inject(r, h, lam=0.0)
    np.testing.assert_array_equal(out, h)
    # h = 0, lambda = 2^k: out = 2^k * m exactly (a power-of-two scaling of a bf16 is a bf16)
    z = np.zeros_like(h)
    for k in (-3, 0, 4):
        _, out = o.inject(r, z, lam=2.0 ** k)
        np.testing.assert_array_equal(unbf(out[1]), unbf(bf(m)) * 2.0 ** k)
    # m = h, lambda = 1: out = 2h exactly
    hh = np.stack([h[0], bf(m), h[2]])
    _, out = o.inject(r, hh, lam=1.0)
    np.testing.assert_array_equal(unbf(out[1]), 2 * unbf(bf(m)))
    # all-zero rows: identity
    o0, _ = _one_hit_oracle(oracle_mod, np.zeros(d), d=d)
    _, out = o0.inject(o0.lookup(tok), h, lam=3.0)
    np.testing.assert_array_equal(unbf(out), unbf(h))
    # matched but not GPU-resident: identity, bitwise, and listed as a miss
    for state, tier in ((-1, 2), (-2, 3)):
        om, _ = _one_hit_oracle(oracle_mod, m, d=d, state=state)
        rm = om.lookup(tok)
        _, out = om.inject(rm, h, lam=1.0)
        np.testing.assert_array_equal(out, h)
        assert list(zip(rm.miss_q, rm.miss_phrase, rm.miss_tier)) == [(1, 0, tier)]
        assert rm.sel_slot.tolist() == [-3, state, -3]


def test_injection_fp32_hidden(oracle_mod):
    d = 8
    row = [0.5, -0.25, 2.0, 0.0, 1.0, 0.1, 0.2, -1.5]
    o, tok = _one_hit_oracle(oracle_mod, row)
    h = np.linspace(-1, 1, 3 * d).astype(np.float32).reshape(3, d)
    r = o.lookup(tok)
    exact, out = o.inject(r, h, lam=0.3, hidden_dtype=oracle_mod.HIDDEN_F32)
    want = h[1].astype(np.float64) + 0.3 * unbf(bf(row))
    np.testing.assert_allclose(exact[1], want, rtol=0, atol=1e-15)
    np.testing.assert_array_equal(out[1], want.astype(np.float32))
    np.testing.assert_array_equal(out[[0, 2]], h[[0, 2]])


# --------------------------------------------------------------- aggregation


def _two_match_oracle(oracle_mod, r2, r3, s2=0, s3=1, d=4):
    rows = np.zeros((2, d), np.uint16)
    if s2 >= 0:
        rows[s2] = bf(r2)
    if s3 >= 0:
        rows[s3] = bf(r3)
    o = mk_oracle(oracle_mod, [(2, 3), (1, 2, 3)], [s2, s3], rows, d, 10, [2, 3], 2)
    return o, np.array([[1, 2, 3]], np.int32)


def test_all_policy_weights_by_length(oracle_mod):
    A = oracle_mod.POLICY_ALL
    o, tok = _two_match_oracle(oracle_mod, [5.0, 0.0, -10.0, 2.5], [10.0, 5.0, 0.0, -2.5])
    h = bf(np.array([[0, 0, 0, 0], [0, 0, 0, 0], [1.0, 1.0, 1.0, 1.0]], np.float32))
    r = o.lookup(tok, 0, A)
    exact, out = o.inject(r, h, policy=A, lam=0.5)
    # alpha = 2/5 and 3/5:  m = (2+6, 0+3, -4+0, 1-1.5) = (8, 3, -4, -0.5);  out = 1 + 0.5 m
    np.testing.assert_allclose(exact[2], [5.0, 2.5, -1.0, 0.75], rtol=0, atol=1e-12)
    np.testing.assert_array_equal(unbf(out[2]), [5.0, 2.5, -1.0, 0.75])
    np.testing.assert_array_equal(out[:2], h[:2])
    # identical vectors: the weights sum to one, m = e
    o, tok = _two_match_oracle(oracle_mod, [1.0, 2.0, 3.0, 4.0], [1.0, 2.0, 3.0, 4.0])
    exact, _ = o.inject(o.lookup(tok, 0, A), h, policy=A, lam=1.0)
    np.testing.assert_allclose(exact[2], [2.0, 3.0, 4.0, 5.0], rtol=0, atol=1e-12)
    # a matched but non-resident member keeps its weight share and is listed as a miss
    o, tok = _two_match_oracle(oracle_mod, [5.0, 0.0, -10.0, 2.5], None, s2=0, s3=-1)
    r = o.lookup(tok, 0, A)
    exact, _ = o.inject(r, h, policy=A, lam=0.5)
    np.testing.assert_allclose(exact[2], [2.0, 1.0, -1.0, 1.5], rtol=0, atol=1e-12)
    assert list(zip(r.miss_q, r.miss_phrase, r.miss_tier)) == [(2, 1, 2)]
    # LONGEST on the same table selects the host-resident 3-gram: no injection at all
    rl = o.lookup(tok, 0)
    _, out = o.inject(rl, h, lam=0.5)
    np.testing.assert_array_equal(out, h)


def test_all_policy_single_match_reduces_to_longest(oracle_mod):
    rng = np.random.default_rng(11)
    d = 16
    rows = bf(rng.standard_normal((1, d)))
    o = mk_oracle(oracle_mod, [(4, 5)], [0], rows, d, 10, [2, 3], 1)
    tok = np.array([[3, 4, 5, 4, 5]], np.int32)
    h = bf(rng.standard_normal((5, d)))
    rl, ra = o.lookup(tok), o.lookup(tok, 0, oracle_mod.POLICY_ALL)
    el, ol = o.inject(rl, h, lam=0.7)
    ea, oa = o.inject(ra, h, policy=oracle_mod.POLICY_ALL, lam=0.7)
    np.testing.assert_array_equal(ol, oa)
    np.testing.assert_allclose(el, ea, rtol=0, atol=1e-15)


# --------------------------------------------------------------- cosine gate


def test_cosine_gate_special_cases(oracle_mod):
    d = 8
    G = oracle_mod.GATE_COSINE
    hv = np.array([1.0, -2.0, 0.5, 0.25, 0.0, 1.5, -1.0, 2.0], np.float32)
    sig = lambda x: 1.0 / (1.0 + np.exp(-x))
    lam = 0.8
    cases = {
        "m=h": (hv, lam * sig(1.0)),
        "m=-h": (-hv, lam * sig(-1.0)),
        "m orthogonal": (np.array([2.0, 1.0, 0, 0, 5.0, 0, 0, 0], np.float32), lam * 0.5),
    }
    for name, (mv, g) in cases.items():
        o, tok = _one_hit_oracle(oracle_mod, mv, d=d)
        h = bf(np.stack([hv, hv, hv]))
        exact, _ = o.inject(o.lookup(tok), h, gate=G, lam=lam)
        np.testing.assert_allclose(exact[1], hv.astype(np.float64) + g * mv.astype(np.float64),
                                   rtol=0, atol=1e-9, err_msg=name)
    o, tok = _one_hit_oracle(oracle_mod, np.zeros(d), d=d)
    h = bf(np.stack([hv, hv, hv]))
    _, out = o.inject(o.lookup(tok), h, gate=G, lam=lam)
    np.testing.assert_array_equal(unbf(out), unbf(h))


# ------------------------------------------------ tiers, miss list, install


def _small_workload(oracle_mod, residency="hot_host_ssd", seed=9, N=1500, C=600, policy_orders=(2, 3)):
    w = synth.config(1, seed=seed, n_phrases=N, gpu_slots=C, residency=residency, d=32, B=6, T=40,
                     p=0.45, orders=tuple(policy_orders))
    tb = synth.make_table(w)
    rows = synth.make_rows_np(w, tb)
    o = oracle_mod.Oracle(tb.phrase_tokens, tb.phrase_len, tb.init_slot, rows, d=w.d, vocab=w.vocab,
                          orders=w.orders, gpu_slots=w.gpu_slots)
    return w, tb, o


@pytest.mark.parametrize("policy", [0, 1])
def test_tier_and_miss_list_invariants(oracle_mod, policy):
    w, tb, o = _small_workload(oracle_mod)
    tok = synth.make_queries(w, tb)
    r = o.lookup(tok, 0, policy)
    f = r.flags.ravel()
    assert np.bincount(f, minlength=4).sum() == f.size
    assert len(r.miss_q) == np.count_nonzero(f >= 2) > 0
    assert np.count_nonzero(f == 1) > 0
    # listed phrases are exactly the non-resident retained ones, in ascending (q, order)
    assert np.all(o.slot_state[r.miss_phrase] < 0)
    np.testing.assert_array_equal(r.miss_tier, np.where(o.slot_state[r.miss_phrase] == -1, 2, 3))
    if policy == 0:
        assert np.all(np.diff(r.miss_q.astype(np.int64)) > 0)
        np.testing.assert_array_equal(r.miss_q, np.nonzero(f >= 2)[0])
        np.testing.assert_array_equal(r.miss_phrase, r.sel_phrase[f >= 2])
    else:
        qq, oo = np.nonzero(r.flags >= 2)
        np.testing.assert_array_equal(r.miss_q, qq)
        np.testing.assert_array_equal(r.miss_phrase, r.sel_phrase[qq, oo])
    # GPU hits point at the slot that holds that phrase
    hit = f == 1
    np.testing.assert_array_equal(o.slot_owner[r.sel_slot.ravel()[hit]], r.sel_phrase.ravel()[hit])


def test_install_converges_to_the_all_resident_result(oracle_mod):
    w, tb, o = _small_workload(oracle_mod, N=1200, C=1200, residency="hot_host_ssd")
    # start with only 400 resident: rebuild residency by hand
    w2 = synth.config(1, seed=9, n_phrases=1200, gpu_slots=1200, residency="hot_host_ssd",
                      reserve_free=800, d=32, B=6, T=40, p=0.45)
    tb2 = synth.make_table(w2)
    rows2 = synth.make_rows_np(w2, tb2)
    o2 = oracle_mod.Oracle(tb2.phrase_tokens, tb2.phrase_len, tb2.init_slot, rows2, d=32,
                           vocab=w2.vocab, orders=w2.orders, gpu_slots=1200)
    tok = synth.make_queries(w2, tb2)
    h = synth.make_hidden_np(w2)
    r = o2.lookup(tok)
    assert len(r.miss_q) > 0
    ids = np.unique(r.miss_phrase)
    free = np.nonzero(o2.slot_owner < 0)[0][:len(ids)].astype(np.int32)
    assert o2.cache_install(ids, synth.phrase_rows_np(w2, ids), free) == 0
    r2 = o2.lookup(tok)
    assert len(r2.miss_q) == 0
    np.testing.assert_array_equal(r2.sel_phrase, r.sel_phrase)
    # reference: the same table with every phrase resident from the start (other slots)
    wall = synth.config(1, seed=9, n_phrases=1200, gpu_slots=1200, residency="all", d=32, B=6, T=40,
                        p=0.45)
    tball = synth.make_table(wall)
    oall = oracle_mod.Oracle(tball.phrase_tokens, tball.phrase_len, tball.init_slot,
                             synth.make_rows_np(wall, tball), d=32, vocab=wall.vocab,
                             orders=wall.orders, gpu_slots=1200)
    rall = oall.lookup(tok)
    np.testing.assert_array_equal(rall.sel_phrase, r2.sel_phrase)     # slot permutation changes slots only
    np.testing.assert_array_equal(rall.flags, r2.flags)
    _, out_a = oall.inject(rall, h, lam=1.0)
    _, out_b = o2.inject(r2, h, lam=1.0)
    np.testing.assert_array_equal(out_a, out_b)


def test_cache_install_state_machine(oracle_mod):
    d = 4
    rows = np.zeros((3, d), np.uint16)
    rows[0] = bf([1, 1, 1, 1])
    rows[1] = bf([2, 2, 2, 2])
    phrases = [(1, 2), (2, 3), (3, 4), (4, 5)]
    o = mk_oracle(oracle_mod, phrases, [0, 1, -1, -2], rows, d, 10, [2], 3)
    before = (o.slot_state.copy(), o.slot_owner.copy(), o.rows.copy())
    src = bf(np.array([[7, 7, 7, 7], [8, 8, 8, 8]], np.float32))
    # refusals leave everything untouched
    assert o.cache_install([9, 2], src, [2, 1]) == -1      # unknown phrase
    assert o.cache_install([0, 2], src, [2, 1]) == -2      # already resident
    assert o.cache_install([2, 3], src, [2, 3]) == -3      # slot out of range
    assert o.cache_install([2, 2], src, [2, 1]) == -4      # repeated id
    assert o.cache_install([2, 3], src, [2, 2]) == -5      # repeated slot
    for a, b in zip(before, (o.slot_state, o.slot_owner, o.rows)):
        np.testing.assert_array_equal(a, b)
    # phrase 2 -> free slot 2; phrase 3 -> slot 1, evicting phrase 1 to the host tier
    assert o.cache_install([2, 3], src, [2, 1]) == 0
    assert o.slot_state.tolist() == [0, -1, 2, 1]
    assert o.slot_owner.tolist() == [0, 3, 2]
    np.testing.assert_array_equal(o.rows[2], src[0])
    np.testing.assert_array_equal(o.rows[1], src[1])
    tok = np.array([[1, 2, 3, 4, 5]], np.int32)
    r = o.lookup(tok)
    assert r.flags.tolist() == [0, 1, 2, 1, 1]
    assert r.sel_slot.tolist() == [-3, 0, -1, 2, 1]
    assert list(zip(r.miss_q, r.miss_phrase, r.miss_tier)) == [(2, 1, 2)]


# ------------------------------------------------------ the paper's Table 1


def test_paper_table_hash_occupancy_fixture():
    rows = []
    with open(os.path.join(GOLDEN, "hash_occupancy.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            M, B, avg = line.split()
            rows.append((int(M), int(B), float(avg)))
    assert len(rows) == 3
    for M, B, avg in rows:
        assert M / B == avg
        occupied = B * (1.0 - (1.0 - 1.0 / B) ** M)
        assert 0 < occupied <= B
    # M = B: a fraction 1 - 1/e of the slots is occupied
    M, B, _ = rows[0]
    assert abs(B * (1.0 - (1.0 - 1.0 / B) ** M) / B - (1 - np.exp(-1))) < 1e-6


# ------------------------------------------- prefetch candidates + priority


def _py_prefetch(phrases, state, history, cand, prob, vocab, orders, use, c_host, c_ssd, budget):
    """Independent restatement: dict matcher, float32 products, python sort."""
    table = {tuple(int(x) for x in p): i for i, p in enumerate(phrases)}
    B, H = history.shape
    K = cand.shape[1]
    out = []
    for b in range(B):
        for k in range(K):
            for oi, n in enumerate(orders):
                if n - 1 > H:
                    continue
                g = tuple(int(x) for x in history[b, H - (n - 1):]) + (int(cand[b, k]),) if n > 1 else (int(cand[b, k]),)
                if not all(0 <= x < vocab for x in g) or g not in table:
                    continue
                i = table[g]
                if state[i] >= 0:
                    continue
                c = np.float32(c_host if state[i] == -1 else c_ssd)
                r = np.float32(1.0 if use is None else use[i])
                s = np.float32(np.float32(np.float32(prob[b, k]) * r) * c)
                if not s > 0:
                    continue
                out.append((-float(s), (b * K + k) * len(orders) + oi, i, 2 if state[i] == -1 else 3, b * K + k))
    out.sort()
    return out[:budget], len(out)


def test_prefetch_candidates_by_hand(oracle_mod):
    # history "... 10 11", predicted next tokens 12 (p=.5), 13 (p=.3), 14 (p=.2)
    phrases = [(11, 12), (10, 11, 12), (11, 13), (11, 14), (10, 11, 14), (12,)]
    state = [-2, -1, 0, -1, -2, -1]           # SSD, host, GPU-resident, host, SSD, host
    o = mk_oracle(oracle_mod, phrases, state, np.zeros((1, 8), np.uint16), 8, 100, [2, 3], 1)
    hist = np.array([[10, 11]], np.int32)
    cand = np.array([[12, 13, 14]], np.int32)
    prob = np.array([[0.5, 0.3, 0.2]], np.float32)
    use = np.array([1.0, 2.0, 1.0, 4.0, 1.0, 1.0], np.float32)
    ph, tr, sc, src, total = o.prefetch_candidates(hist, cand, prob, usefulness=use, benefit_host=1.0, benefit_ssd=2.0,
                                                   budget=10)
    # (11,12) SSD: .5*1*2 = 1.0 ; (10,11,12) host: .5*2*1 = 1.0 (same priority, later order) ; (11,13) is
    # GPU-resident: no candidate ; (11,14) host: .2*4*1 = .8 ; (10,11,14) SSD: .2*1*2 = .4 ; (12,) is an
    # order-1 phrase but order 1 is not configured
    assert total == 4
    assert ph.tolist() == [0, 1, 3, 4] and tr.tolist() == [3, 2, 2, 3] and src.tolist() == [0, 0, 2, 2]
    np.testing.assert_array_equal(sc, np.array([1.0, 1.0, np.float32(0.2) * np.float32(4.0), np.float32(np.float32(0.2) * 1) * 2],
                                               np.float32))
    # budget cut keeps the best
    ph2, _, _, _, total2 = o.prefetch_candidates(hist, cand, prob, usefulness=use, budget=2)
    assert total2 == 4 and ph2.tolist() == [0, 1]
    # no usefulness table: r = 1
    ph3, _, sc3, _, _ = o.prefetch_candidates(hist, cand, prob, budget=10)
    assert ph3.tolist() == [0, 1, 4, 3]       # 1.0, 0.5, 0.4, 0.2
    # zero benefit for the host tier drops host-resident candidates
    ph4, tr4, _, _, total4 = o.prefetch_candidates(hist, cand, prob, benefit_host=0.0, budget=10)
    assert total4 == 2 and set(tr4.tolist()) == {3}


@pytest.mark.parametrize("seed,orders", [(1, [2, 3]), (2, [1, 2, 3, 4]), (3, [3])])
def test_prefetch_candidates_against_python_restatement(oracle_mod, seed, orders):
    rng = np.random.default_rng(seed)
    V = 7
    phrases = set()
    target = min(250, sum(V ** n for n in orders) // 2)
    while len(phrases) < target:
        n = int(rng.choice(orders))
        phrases.add(tuple(int(x) for x in rng.integers(0, V, n)))
    phrases = sorted(phrases, key=lambda p: rng.random())
    state = rng.choice([-2, -1, 5], size=len(phrases)).astype(np.int32)
    state[state == 5] = np.arange((state == 5).sum())
    o = mk_oracle(oracle_mod, phrases, state, np.zeros((len(phrases), 8), np.uint16), 8, V, orders, len(phrases))
    B, H, K = 6, 3, 9
    hist = rng.integers(-1, V + 1, size=(B, H)).astype(np.int32)
    cand = rng.integers(-1, V + 1, size=(B, K)).astype(np.int32)
    prob = rng.random((B, K)).astype(np.float32)
    prob[rng.random((B, K)) < 0.2] = np.float32(0.25)       # ties
    use = rng.choice([0.5, 1.0, 2.0, 0.0], size=len(phrases)).astype(np.float32)
    for budget in (5, 10_000):
        ph, tr, sc, src, total = o.prefetch_candidates(hist, cand, prob, usefulness=use, benefit_host=1.0,
                                                       benefit_ssd=1.5, budget=budget)
        exp, exp_total = _py_prefetch(phrases, state, hist, cand, prob, V, orders, use, 1.0, 1.5, budget)
        assert total == exp_total > 5
        assert ph.tolist() == [e[2] for e in exp]
        assert tr.tolist() == [e[3] for e in exp]
        assert src.tolist() == [e[4] for e in exp]
        np.testing.assert_array_equal(sc, np.array([-e[0] for e in exp], np.float32))


# ---------------------------------------------------------------- retention ranking (Sec. 4.3)

def _mini_oracle(orc, C, owners=None):
    """An oracle over C single-slot phrases (phrase i lives in slot i unless owners says otherwise)."""
    N = C
    pt = np.full((N, 4), -1, np.int32)
    pt[:, 0] = np.arange(N) // 50
    pt[:, 1] = np.arange(N) % 50
    pl = np.full(N, 2, np.uint8)
    init = np.arange(N, dtype=np.int32) if owners is None else np.asarray(owners, np.int32)
    rows = np.zeros((C, 16), np.uint16)
    return orc.Oracle(pt, pl, init, rows, d=16, vocab=64, orders=(2,), gpu_slots=C)


def test_retention_key_hand_worked(oracle_mod):
    k = oracle_mod.lib().orc_retention_key
    # no decay: frequency in the high half, 65535 - age in the low half
    assert k(3, 10, 12, 0) == (3 << 16) | (65535 - 2)
    # half-life 4, idle for 9 epochs: two halvings of 13 -> 3
    assert k(13, 1, 10, 4) == (3 << 16) | (65535 - 9)
    # saturation of both halves; shift capped at 31
    assert k(1 << 20, 5, 5, 0) == (65535 << 16) | 65535
    assert k(7, 0, 100000, 0) == (7 << 16) | 0
    assert k(0xFFFFFFFF, 0, 1000, 1) == (1 << 16) | (65535 - 1000)
    # monotone: more hits never lowers the key; longer idle never raises it
    for f in range(0, 40):
        assert k(f + 1, 3, 9, 2) >= k(f, 3, 9, 2)
        assert k(20, 3, 9 + f + 1, 2) <= k(20, 3, 9 + f, 2)


def test_retention_reduces_to_lru_and_lfu(oracle_mod):
    rng = np.random.default_rng(5)
    C = 64
    o = _mini_oracle(oracle_mod, C)
    # equal frequencies, distinct last-use epochs: victims come in least-recently-used order
    o.freq[:] = 1
    o.last[:] = rng.permutation(C).astype(np.uint32)
    o.epoch = C
    slots, _ = o.cache_victims(10, half_life=0)
    np.testing.assert_array_equal(slots, np.argsort(o.last, kind="stable")[:10])
    # equal last use, distinct frequencies: least-frequently-used order
    o.last[:] = 7
    o.freq[:] = (rng.permutation(C) + 1).astype(np.uint32)
    slots, _ = o.cache_victims(C + 5, half_life=0)
    np.testing.assert_array_equal(slots, np.argsort(o.freq, kind="stable"))
    # ties keep ascending slot order
    o.freq[:] = 2
    slots, keys = o.cache_victims(5)
    np.testing.assert_array_equal(slots, np.arange(5))
    assert len(set(keys.tolist())) == 1


def test_retention_free_slots_first_and_state_updates(oracle_mod):
    C = 12
    owners = np.arange(C, dtype=np.int32)
    owners[[3, 8]] = -1                      # phrases 3 and 8 start on the host: slots 3 and 8 are free
    o = _mini_oracle(oracle_mod, C, owners)
    toks = np.array([[0, 0, 0, 1, 0, 1, 0, 5]], np.int32)     # 2-grams (0,0) (0,0) (0,1) (1,0) (0,1) (1,0) (0,5)
    res = o.lookup(toks)
    o.touch(res)                              # epoch 0 -> 1
    res2 = o.lookup(np.array([[0, 1, 0, 0]], np.int32))
    o.touch(res2)                             # epoch 1 -> 2
    # phrase ids: (0,0)=0, (0,1)=1, (0,5)=5, (1,0)=50 (not in this 12-phrase table)
    expect_freq = np.zeros(C, np.uint32); expect_last = np.zeros(C, np.uint32)
    expect_freq[0], expect_last[0] = 3, 1     # (0,0): twice in call 0, once in call 1
    expect_freq[1], expect_last[1] = 3, 1     # (0,1): twice in call 0, once in call 1
    expect_freq[5], expect_last[5] = 1, 0
    np.testing.assert_array_equal(o.freq, expect_freq)
    np.testing.assert_array_equal(o.last, expect_last)
    assert o.epoch == 2
    slots, keys = o.cache_victims(4)
    # free slots (key 0) first in slot order, then never-used owned slots: age 2, freq 0
    np.testing.assert_array_equal(slots, [3, 8, 2, 4])
    np.testing.assert_array_equal(keys, [0, 0, 65533, 65533])
    # installing phrase 3 into slot 8 makes the slot owned, used once, now
    assert o.cache_install([3], np.ones((1, 16), np.uint16), [8]) == 0
    assert o.freq[8] == 1 and o.last[8] == 2
    slots, _ = o.cache_victims(C)
    assert slots[0] == 3 and list(slots).index(8) > list(slots).index(5) > list(slots).index(4)
    assert slots[-1] == 1 and slots[-2] == 0


def test_retention_against_independent_restatement(oracle_mod):
    rng = np.random.default_rng(11)
    C = 5000
    owners = np.arange(C, dtype=np.int32)
    owners[rng.choice(C, 37, replace=False)] = -1
    o = _mini_oracle(oracle_mod, C, owners)
    o.freq[:] = rng.geometric(0.02, C).astype(np.uint32) * (rng.random(C) < 0.8)
    o.freq[rng.choice(C, 5)] = 3_000_000
    o.epoch = 90_000
    o.last[:] = (o.epoch - np.minimum(o.epoch, rng.geometric(0.0005, C))).astype(np.uint32)
    for hl in (0, 1, 7, 300, 100_000):
        age = (np.uint64(o.epoch) - o.last.astype(np.uint64))
        shift = np.minimum(31, age // hl) if hl > 0 else np.zeros(C, np.uint64)
        dec = np.minimum(o.freq.astype(np.uint64) >> shift.astype(np.uint64), 65535)
        key = (dec << np.uint64(16)) | (np.uint64(65535) - np.minimum(age, 65535))
        key[o.slot_owner < 0] = 0
        order = np.lexsort((np.arange(C), key))
        slots, keys = o.cache_victims(700, half_life=hl)
        np.testing.assert_array_equal(slots, order[:700])
        np.testing.assert_array_equal(keys, key[order[:700]].astype(np.uint32))


# ---------------------------------------------------------------- early-exit prefetch head (Sec. 4.4)

def test_head_hand_worked(oracle_mod):
    # W rows pick out single coordinates of h, so the logits are the entries of h: ln 1 .. ln 4 (rounded
    # to bf16) and the distribution is (almost) 0.1, 0.2, 0.3, 0.4
    lg = unbf(bf(np.log([1.0, 2.0, 3.0, 4.0])))
    W = bf(np.eye(4))
    h = bf(np.log([[1.0, 2.0, 3.0, 4.0]]))
    z = oracle_mod.head_logits(W, h)
    np.testing.assert_array_equal(z, lg[None, :])
    tok, prob, lse = oracle_mod.head_topk(z, 3)
    np.testing.assert_array_equal(tok, [[3, 2, 1]])
    expect = np.exp(lg) / np.exp(lg).sum()
    np.testing.assert_allclose(prob[0], expect[[3, 2, 1]], rtol=1e-14)
    np.testing.assert_allclose(prob[0], [0.4, 0.3, 0.2], atol=2e-3)       # bf16 rounding of the logs
    np.testing.assert_allclose(lse[0], np.log(np.exp(lg).sum()), rtol=1e-14)


def test_head_against_library_routines(oracle_mod):
    rng = np.random.default_rng(3)
    V, d, B, K = 3000, 96, 5, 17
    W = bf(rng.standard_normal((V, d)) * 0.3)
    h = bf(rng.standard_normal((B, d)))
    z = oracle_mod.head_logits(W, h)
    zt = torch.from_numpy(unbf(h)) @ torch.from_numpy(unbf(W)).T                 # float64 matmul
    np.testing.assert_allclose(z, zt.numpy(), rtol=0, atol=1e-12)
    tok, prob, lse = oracle_mod.head_topk(z, K)
    p = torch.softmax(torch.from_numpy(z), dim=1)
    pv, pi = torch.topk(p, K, dim=1)
    np.testing.assert_array_equal(tok, pi.numpy())
    np.testing.assert_allclose(prob, pv.numpy(), rtol=1e-12)
    np.testing.assert_allclose(lse, torch.logsumexp(torch.from_numpy(z), dim=1).numpy(), rtol=1e-13)
    # all of it sums to one
    _, pall, _ = oracle_mod.head_topk(z, V)
    np.testing.assert_allclose(pall.sum(axis=1), 1.0, rtol=1e-12)


def test_head_invariants(oracle_mod):
    rng = np.random.default_rng(4)
    V, d = 500, 32
    W = bf(rng.standard_normal((V, d)))
    h = bf(rng.standard_normal((3, d)))
    z = oracle_mod.head_logits(W, h)
    tok, prob, _ = oracle_mod.head_topk(z, 8)
    # h = 0: uniform distribution, ties resolved by ascending token id
    t0, p0, l0 = oracle_mod.head_topk(oracle_mod.head_logits(W, np.zeros((1, d), np.uint16)), 5)
    np.testing.assert_array_equal(t0, [[0, 1, 2, 3, 4]])
    np.testing.assert_allclose(p0, 1.0 / V, rtol=1e-14)
    np.testing.assert_allclose(l0, np.log(V), rtol=1e-14)
    # permuting the rows of W permutes the token ids and nothing else
    perm = rng.permutation(V)
    tp, pp, _ = oracle_mod.head_topk(oracle_mod.head_logits(W[perm], h), 8)
    np.testing.assert_array_equal(perm[tp], tok)
    np.testing.assert_allclose(pp, prob, rtol=1e-12)        # the sum runs in another order
    # a constant added to every logit changes no probability
    t2, p2, _ = oracle_mod.head_topk(z + 7.5, 8)
    np.testing.assert_array_equal(t2, tok)
    np.testing.assert_allclose(p2, prob, rtol=1e-12)
    # duplicate rows of W tie exactly: the lower id comes first
    W2 = W.copy(); W2[10] = W2[400]
    z2 = oracle_mod.head_logits(W2, h)
    t3, _, _ = oracle_mod.head_topk(z2, V)
    for b in range(3):
        pos = {int(v): i for i, v in enumerate(t3[b])}
        assert pos[400] == pos[10] + 1


# ---------------------------------------------------------------- lenient installation

def test_lenient_install_hand_worked(oracle_mod):
    # 8 phrases (i // 50, i % 50), 5 slots; phrases 0, 1, 2 start in slots 0, 1, 2; slots 3, 4 are free
    owners = np.array([0, 1, 2, -1, -1, -1, -2, -1], np.int32)
    pt = np.full((8, 4), -1, np.int32); pt[:, 0] = 0; pt[:, 1] = np.arange(8)
    o = oracle_mod.Oracle(pt, np.full(8, 2, np.uint8), owners, np.zeros((5, 16), np.uint16), d=16, vocab=64,
                          orders=(2,), gpu_slots=5)
    ids = np.array([3, 9, 1, 4, 3, 5, 6, 7, 7], np.uint32)
    dst = np.array([3, 4, 4, 3, 4, 7, 1, -1, 0], np.int32)
    src = (np.arange(9)[:, None] + 1).astype(np.uint16) * np.ones((1, 16), np.uint16)
    applied, cnt = o.cache_install_lenient(ids, src, dst)
    # 0: phrase 3 -> free slot 3: applied.          1: id 9 is no phrase.            2: phrase 1 is resident.
    # 3: phrase 4 -> slot 3, taken by entry 0.      4: phrase 3 again.               5: slot 7 does not exist.
    # 6: phrase 6 (SSD) -> slot 1, evicts phrase 1. 7: slot -1 does not exist.       8: phrase 7 again (entry 7 came first).
    np.testing.assert_array_equal(applied, [1, 0, 0, 0, 0, 0, 1, 0, 0])
    assert cnt == 2
    np.testing.assert_array_equal(o.slot_state, [0, -1, 2, 3, -1, -1, 1, -1])
    np.testing.assert_array_equal(o.slot_owner, [0, 6, 2, 3, -1])
    assert (o.rows[3] == 1).all() and (o.rows[1] == 7).all() and (o.rows[0] == 0).all()


def test_lenient_install_equals_strict_install_on_clean_batches(oracle_mod):
    rng = np.random.default_rng(12)
    for trial in range(20):
        N, C = 300, 120
        owners = np.full(N, -1, np.int32)
        res = rng.choice(N, 80, replace=False)
        owners[res] = rng.permutation(C)[:80]
        pt = np.full((N, 4), -1, np.int32); pt[:, 0] = np.arange(N) // 20; pt[:, 1] = np.arange(N) % 20
        mk = lambda: oracle_mod.Oracle(pt, np.full(N, 2, np.uint8), owners, np.zeros((C, 8), np.uint16), d=8, vocab=32,
                                       orders=(2,), gpu_slots=C)
        a, b = mk(), mk()
        n = int(rng.integers(1, 60))
        ids = rng.choice(np.nonzero(owners < 0)[0], n, replace=False).astype(np.uint32)
        dst = rng.choice(C, n, replace=False).astype(np.int32)
        src = rng.integers(1, 60000, size=(n, 8)).astype(np.uint16)
        assert a.cache_install(ids, src, dst) == 0
        applied, cnt = b.cache_install_lenient(ids, src, dst)
        assert cnt == n and applied.all()
        np.testing.assert_array_equal(a.slot_state, b.slot_state)
        np.testing.assert_array_equal(a.slot_owner, b.slot_owner)
        np.testing.assert_array_equal(a.rows, b.rows)


def test_lenient_install_against_independent_restatement(oracle_mod):
    rng = np.random.default_rng(13)
    for trial in range(30):
        N, C = 200, 64
        owners = np.full(N, -1, np.int32)
        res = rng.choice(N, 40, replace=False)
        owners[res] = rng.permutation(C)[:40]
        owners[rng.choice(np.nonzero(owners < 0)[0], 30, replace=False)] = -2
        pt = np.full((N, 4), -1, np.int32); pt[:, 0] = np.arange(N) // 20; pt[:, 1] = np.arange(N) % 20
        o = oracle_mod.Oracle(pt, np.full(N, 2, np.uint8), owners, np.zeros((C, 4), np.uint16), d=4, vocab=32,
                              orders=(2,), gpu_slots=C)
        n = int(rng.integers(1, 150))
        ids = rng.integers(0, N + 20, size=n).astype(np.uint32)
        dst = rng.integers(-3, C + 5, size=n).astype(np.int32)
        src = (np.arange(n)[:, None] + 1).astype(np.uint16) * np.ones((1, 4), np.uint16)
        # restatement with dictionaries and sets
        state = {i: int(owners[i]) for i in range(N)}
        owner = {int(owners[i]): i for i in range(N) if owners[i] >= 0}
        rows = {}
        seen_ids, seen_slots, expect = set(), set(), []
        for k in range(n):
            i, s_ = int(ids[k]), int(dst[k])
            cand = i < N and owners[i] < 0 and 0 <= s_ < C and i not in seen_ids
            seen_ids.add(i)
            ok = cand and s_ not in seen_slots
            if cand:
                seen_slots.add(s_)
            expect.append(int(ok))
        for k in range(n):
            if expect[k]:
                i, s_ = int(ids[k]), int(dst[k])
                if s_ in owner:
                    state[owner[s_]] = -1
                state[i] = s_; owner[s_] = i; rows[s_] = k + 1
        applied, cnt = o.cache_install_lenient(ids, src, dst)
        np.testing.assert_array_equal(applied, expect)
        assert cnt == sum(expect)
        np.testing.assert_array_equal(o.slot_state, [state[i] for i in range(N)])
        np.testing.assert_array_equal(o.slot_owner, [owner.get(s_, -1) for s_ in range(C)])
        for s_, v in rows.items():
            assert (o.rows[s_] == v).all()


# ---------------------------------------------------------------------------------------------
# n-gram extraction with a frequency threshold (Sec. 4.2 construction pipeline, Sec. 5.3)
# ---------------------------------------------------------------------------------------------
def test_mine_ngrams_hand_worked(oracle_mod):
    """Corpus 5 7 5 7 9 | 5 7 with one separator, orders 2 and 3, worked by hand: (5,7) ends at 1, 3 and 7;
    the windows ending at 5, 6 (and, for order 3, 7) contain the separator."""
    tok = np.array([5, 7, 5, 7, 9, -1, 5, 7], np.int32)
    pt, pl, pc, n_found, distinct, hist = oracle_mod.mine_ngrams(tok, 10, (2, 3), min_count=1, hist_bins=8)
    assert n_found == 6 and distinct.tolist() == [3, 3]
    assert pt.tolist() == [[5, 7, -1, -1], [7, 5, -1, -1], [5, 7, 5, -1], [7, 5, 7, -1], [7, 9, -1, -1], [5, 7, 9, -1]]
    assert pl.tolist() == [2, 2, 3, 3, 2, 3] and pc.tolist() == [3, 1, 1, 1, 1, 1]
    assert hist.tolist() == [0, 5, 0, 1, 0, 0, 0, 0]
    pt, pl, pc, n_found, _, _ = oracle_mod.mine_ngrams(tok, 10, (2, 3), min_count=2)
    assert n_found == 1 and pt.tolist() == [[5, 7, -1, -1]] and pc.tolist() == [3]
    pt, pl, pc, n_found, _, _ = oracle_mod.mine_ngrams(tok, 10, (2, 3), min_count=1, cap=2)
    assert n_found == 6 and pt.tolist() == [[5, 7, -1, -1], [7, 5, -1, -1]]
    # an id at or above the vocabulary size separates like a negative one; the last histogram bin collects
    pt, _, pc, n_found, distinct, hist = oracle_mod.mine_ngrams(np.array([5, 7, 5, 7, 9, 10, 5, 7], np.int32), 10, (2,), hist_bins=3)
    assert n_found == 3 and pc.tolist() == [3, 1, 1] and hist.tolist() == [0, 2, 1]


def test_mine_ngrams_closed_forms(oracle_mod):
    # one token repeated: a single tuple per order, L - n + 1 times, first met at n - 1
    L = 37
    pt, pl, pc, n_found, distinct, _ = oracle_mod.mine_ngrams(np.full(L, 3, np.int32), 8, (1, 2, 3, 4))
    assert n_found == 4 and pl.tolist() == [1, 2, 3, 4] and pc.tolist() == [L, L - 1, L - 2, L - 3]
    assert distinct.tolist() == [1, 1, 1, 1]
    # a corpus of period P over P different tokens: P tuples per order, the L - n + 1 windows shared out evenly
    P, L = 7, 100
    tok = (np.arange(L) % P).astype(np.int32)
    for n in (2, 3, 4):
        pt, pl, pc, n_found, distinct, _ = oracle_mod.mine_ngrams(tok, P, (n,))
        assert n_found == P == distinct[0] and int(pc.sum()) == L - n + 1
        assert set(pc.tolist()) <= {(L - n + 1) // P, (L - n + 1) // P + 1}
        assert pt[:, 0].tolist() == list(range(P))              # met in corpus order
        assert all(pt[i, j] == (i + j) % P for i in range(P) for j in range(n))
    # every token different: every window is its own tuple, nothing survives a threshold of 2
    tok = np.random.default_rng(5).permutation(500).astype(np.int32)
    pt, pl, pc, n_found, distinct, hist = oracle_mod.mine_ngrams(tok, 500, (2, 3))
    assert n_found == 499 + 498 and distinct.tolist() == [499, 498] and hist[1] == n_found
    assert oracle_mod.mine_ngrams(tok, 500, (2, 3), min_count=2)[3] == 0
    # shorter than the order / empty
    assert oracle_mod.mine_ngrams(np.array([1, 2], np.int32), 5, (3, 4))[3] == 0
    assert oracle_mod.mine_ngrams(np.zeros(0, np.int32), 5, (2,))[3] == 0


@pytest.mark.parametrize("seed", range(6))
def test_mine_ngrams_against_library_unique(oracle_mod, seed):
    """The counts are numpy.unique's over the sliding windows; the order is that of first occurrence."""
    rng = np.random.default_rng([88, seed])
    vocab = int(rng.integers(3, 40))
    L = int(rng.integers(50, 3000))
    tok = rng.integers(0, vocab, size=L).astype(np.int32)
    tok[rng.random(L) < 0.05] = rng.choice([-1, vocab, vocab + 7])
    orders = [o for o in (1, 2, 3, 4) if rng.random() < 0.7] or [2]
    min_count = int(rng.integers(1, 4))
    pt, pl, pc, n_found, distinct, hist = oracle_mod.mine_ngrams(tok, vocab, orders, min_count=min_count, hist_bins=16)
    expect, exp_hist = {}, np.zeros(16, np.int64)
    for oi, n in enumerate(orders):
        win = np.lib.stride_tricks.sliding_window_view(tok, n)                 # window i ends at i + n - 1
        ok = ((win >= 0) & (win < vocab)).all(axis=1)
        uniq, first_idx, counts = np.unique(win[ok], axis=0, return_index=True, return_counts=True)
        ends = np.flatnonzero(ok)[first_idx] + n - 1
        assert distinct[oi] == len(uniq)
        np.add.at(exp_hist, np.minimum(counts, 15), 1)
        for u, e, c in zip(uniq, ends, counts):
            if c >= min_count:
                expect[(int(e), n)] = (tuple(int(x) for x in u), int(c))
    np.testing.assert_array_equal(hist, exp_hist)
    assert n_found == len(expect)
    for i, key in enumerate(sorted(expect)):
        tup, c = expect[key]
        assert pl[i] == key[1] and pc[i] == c
        assert tuple(pt[i, :key[1]].tolist()) == tup and (pt[i, key[1]:] == -1).all()


def test_count_tuple_by_hand_and_against_the_extraction(oracle_mod):
    tok = np.array([5, 7, 5, 7, 9, -1, 5, 7], np.int32)
    assert oracle_mod.count_tuple(tok, (5, 7)) == (3, 1)
    assert oracle_mod.count_tuple(tok, (7, 9)) == (1, 4)
    assert oracle_mod.count_tuple(tok, (9, 5)) == (0, -1)
    assert oracle_mod.count_tuple(tok, (5, 7, 9)) == (1, 4)
    rng = np.random.default_rng(17)
    tok = rng.integers(0, 6, size=4000).astype(np.int32)
    pt, pl, pc, n_found, _, _ = oracle_mod.mine_ngrams(tok, 6, (2, 3, 4))
    for i in rng.choice(n_found, size=40, replace=False):
        n = int(pl[i])
        win = np.lib.stride_tricks.sliding_window_view(tok, n)
        hits = np.flatnonzero((win == pt[i, :n]).all(axis=1))
        assert oracle_mod.count_tuple(tok, pt[i, :n]) == (len(hits), int(hits[0]) + n - 1) == (int(pc[i]), int(hits[0]) + n - 1)


# ---------------------------------------------------------------------------------------------
# initial residency from corpus counts (Sec. 4.3: hottest entries in the GPU tier)
# ---------------------------------------------------------------------------------------------
def test_assign_residency_hand_worked_and_closed_forms(oracle_mod):
    #            id: 0  1  2  3  4  5  6
    count = np.array([5, 9, 5, 1, 9, 2, 5], np.uint32)
    # three slots: the two 9s, then the first of the 5s (id 0); slots in id order: id 0 -> 0, id 1 -> 1, id 4 -> 2
    slot, tiers = oracle_mod.assign_residency(count, 3, host_min_count=2)
    assert slot.tolist() == [0, 1, -1, -2, 2, -1, -1] and tiers == (3, 3, 1)
    slot, tiers = oracle_mod.assign_residency(count, 4, host_min_count=6)
    assert slot.tolist() == [0, 1, 2, -2, 3, -2, -2] and tiers == (4, 0, 3)
    # no slots / more slots than phrases / all counts equal: the first ids
    assert oracle_mod.assign_residency(count, 0, 1)[0].tolist() == [-1] * 7
    assert oracle_mod.assign_residency(count, 100, 1)[0].tolist() == list(range(7))
    assert oracle_mod.assign_residency(np.full(6, 4, np.uint32), 2, 5)[0].tolist() == [0, 1, -2, -2, -2, -2]


@pytest.mark.parametrize("seed", range(5))
def test_assign_residency_against_library_sort(oracle_mod, seed):
    rng = np.random.default_rng([55, seed])
    N = int(rng.integers(1, 5000))
    count = rng.integers(1, int(rng.choice([3, 20, 100000])), size=N).astype(np.uint32)
    G = int(rng.integers(0, N + 5))
    hm = int(rng.integers(0, 6))
    slot, tiers = oracle_mod.assign_residency(count, G, hm)
    order = np.lexsort((np.arange(N), -count.astype(np.int64)))              # count descending, then id
    chosen = np.zeros(N, bool)
    chosen[order[:min(G, N)]] = True
    expect = np.where(count >= hm, -1, -2).astype(np.int32)
    expect[chosen] = np.arange(int(chosen.sum()), dtype=np.int32)
    np.testing.assert_array_equal(slot, expect)
    assert tiers == (int(chosen.sum()), int((expect == -1).sum()), int((expect == -2).sum()))
