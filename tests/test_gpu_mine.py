"""tfe_mine_ngrams (n-gram extraction with a frequency threshold) against the oracle: every output bit-exact."""
import os

import numpy as np
import pytest
import torch

from paper_2607_07388_b200 import synth

pytestmark = pytest.mark.gpu
DEV = torch.device("cuda:0")


@pytest.fixture(scope="module")
def orc():
    from oracle import tfe_oracle
    tfe_oracle.build()
    return tfe_oracle


def _mine_both(orc, tok, vocab, orders, min_count, cap):
    from paper_2607_07388_b200.engine import mine_ngrams
    e_pt, e_pl, e_pc, e_found, e_distinct, e_hist = orc.mine_ngrams(tok, vocab, orders, min_count=min_count, cap=cap)
    got = mine_ngrams(torch.from_numpy(np.ascontiguousarray(tok, np.int32)).to(DEV), vocab=vocab, orders=orders,
                      min_count=min_count, cap=cap)
    assert got.n_found == e_found
    np.testing.assert_array_equal(got.distinct, e_distinct)
    np.testing.assert_array_equal(got.hist, e_hist)
    assert len(got) == len(e_pl)
    np.testing.assert_array_equal(got.phrase_tokens.cpu().numpy(), e_pt)
    np.testing.assert_array_equal(got.phrase_len.cpu().numpy(), e_pl)
    np.testing.assert_array_equal(got.count.cpu().numpy().view(np.uint32), e_pc)
    return got, (e_pt, e_pl, e_pc)


@pytest.mark.parametrize("L", [0, 1, 2, 3, 4, 5, 31, 32, 33, 255, 256, 257, 1023, 1024, 1025, 4097, 20_000])
@pytest.mark.parametrize("vocab", [7, synth.VOCAB])
def test_mine_sizes_and_tails(orc, L, vocab):
    """Lengths around the warp, block and scan-tile sizes; the large vocabulary keys 4-grams through the
    slots of their bigram halves, the small one packs them."""
    rng = np.random.default_rng([3, L, vocab])
    ids = rng.permutation(vocab)[:6]
    tok = ids[rng.integers(0, len(ids), size=L)].astype(np.int32)
    if L:
        tok[rng.random(L) < 0.03] = -1
    for orders in ((2, 3, 4), (4,), (1, 3)):
        _mine_both(orc, tok, vocab, orders, min_count=1, cap=4 * L + 1)
        _mine_both(orc, tok, vocab, orders, min_count=3, cap=4 * L + 1)


@pytest.mark.parametrize("seed", range(int(os.environ.get("TFE_RANDOM_CASES", "16"))))
def test_mine_random(orc, seed):
    rng = np.random.default_rng([4, seed])
    vocab = int(rng.choice([3, 50, 1000, 40_000, synth.VOCAB, 2_000_000]))
    L = int(rng.integers(1, 60_000))
    active = int(rng.integers(2, 300))
    ids = rng.integers(0, vocab, size=active)
    tok = ids[np.minimum(rng.zipf(1.3, size=L) - 1, active - 1)].astype(np.int32)
    sep = rng.random(L) < rng.uniform(0, 0.1)
    tok[sep] = rng.choice([-1, vocab, -5, vocab + 3], size=int(sep.sum()))
    orders = [o for o in (1, 2, 3, 4) if rng.random() < 0.6] or [3]
    min_count = int(rng.integers(0, 6))
    e_found = orc.mine_ngrams(tok, vocab, orders, min_count=min_count, cap=0)[3]
    cap = int(rng.choice([0, 1, max(1, e_found // 2), e_found, e_found + 10]))
    _mine_both(orc, tok, vocab, orders, min_count, cap)


def test_mine_one_hot_tuple(orc):
    """One id repeated: every warp holds 32 equal keys, every atomic lands on one slot."""
    L = 70_001
    for vocab in (9, synth.VOCAB):
        got, _ = _mine_both(orc, np.full(L, vocab - 1, np.int32), vocab, (1, 2, 3, 4), 1, 10)
        assert got.count.cpu().tolist() == [L, L - 1, L - 2, L - 3]


def test_mine_synthetic_corpus_then_build_and_look_up(orc):
    """The construction pipeline end to end on the device: corpus -> phrase table -> index -> lookups, against
    the oracle's table mined from the same corpus and its matcher."""
    import parity_harness as H
    from paper_2607_07388_b200.engine import Engram, bf16_tensor_from_bits
    L, orders, d = 400_000, (2, 3, 4), 64
    corpus = synth.make_corpus(11, L)
    got, (e_pt, e_pl, e_pc) = _mine_both(orc, corpus, synth.VOCAB, orders, min_count=3, cap=L)
    N = len(e_pl)
    assert N > 5_000 and set(np.unique(e_pl).tolist()) == {2, 3, 4}
    # residency: the most frequent half lives in the GPU tier (decided from the oracle's own counts)
    C = N // 2
    order = np.argsort(-e_pc.astype(np.int64), kind="stable")
    init_slot = np.full(N, -1, np.int32)
    init_slot[order[:C]] = np.arange(C, dtype=np.int32)
    init_slot[order[C + (N - C) // 2:]] = -2
    rows = synth.gaussian_bf16([11, 5], (C, d), 1 / 32)
    eng = Engram(got.phrase_tokens, got.phrase_len, torch.from_numpy(init_slot).to(DEV), bf16_tensor_from_bits(rows, DEV),
                 vocab=synth.VOCAB, orders=orders, device_build=True)
    pr = H.Pair.__new__(H.Pair)
    pr.rows_bits, pr.d, pr.C, pr.orders, pr.hidden_dtype, pr.eng = rows, d, C, orders, 0, eng
    pr.ora = orc.Oracle(e_pt, e_pl, init_slot, rows.copy(), d=d, vocab=synth.VOCAB, orders=orders, gpu_slots=C)
    tok = corpus[100_000:100_000 + 4 * 512].reshape(4, 512).copy()          # text the table was mined from: many hits
    h = synth.gaussian_bf16([11, 6], (4 * 512, d), 1.0)
    _, ref, info = pr.run_and_compare(tok, h, lam=1.0)
    assert info["n_hit"] > 300 and info["n_miss"] > 50
    pr.run_and_compare(tok, h, lam=1.0, policy=1)
    pr.close()


def test_mine_histogram_picks_the_threshold(orc):
    """sum_{c >= m} hist[c] is the table size for threshold m: one call, then the threshold for a wanted size."""
    from paper_2607_07388_b200.engine import mine_ngrams
    corpus = torch.from_numpy(synth.make_corpus(12, 300_000)).to(DEV)
    first = mine_ngrams(corpus, vocab=synth.VOCAB, orders=(2, 3), min_count=1, cap=0)
    tail = np.cumsum(first.hist[::-1])[::-1]
    assert tail[1] == first.n_found == first.distinct.sum()
    want = 20_000
    m = int(np.argmax(tail <= want))
    assert 1 < m < 1023
    second = mine_ngrams(corpus, vocab=synth.VOCAB, orders=(2, 3), min_count=m, cap=want, want_hist=False)
    assert second.n_found == tail[m] <= want < tail[m - 1] and len(second) == second.n_found
    assert int(second.count.min()) >= m


def test_mine_workspace_and_argument_checks():
    from paper_2607_07388_b200 import binding as tfe
    assert tfe.tfe_mine_workspace_bytes(1 << 20, 3) >= (1 << 21) * 16
    tok = torch.zeros(16, dtype=torch.int32, device=DEV)
    for orders in ((2, 2), (3, 2), (0,), (5,), (1, 2, 3, 4, 4)):
        with pytest.raises(tfe.TfeError):
            tfe.tfe_mine_ngrams(tok, 16, 10, orders, 1, 0)
    with pytest.raises(tfe.TfeError):
        tfe.tfe_mine_ngrams(tok, -1, 10, (2,), 1, 0)
    with pytest.raises(tfe.TfeError):
        tfe.tfe_mine_ngrams(tok, 16, 0, (2,), 1, 0)
    with pytest.raises(tfe.TfeError):
        tfe.tfe_mine_ngrams(tok, 16, 10, (2,), 1, 4)             # cap > 0 without output arrays
    small = torch.empty(1000, dtype=torch.uint8, device=DEV)
    with pytest.raises(tfe.TfeError) as e:
        tfe.tfe_mine_ngrams(tok, 16, 10, (2,), 1, 0, workspace=small, workspace_bytes=small.numel())
    assert e.value.status == tfe.TFE_ERR_CAPACITY


def test_mine_with_callers_workspace(orc):
    """The same results from a workspace the caller keeps (left dirty between calls, and deliberately misaligned)."""
    from paper_2607_07388_b200 import binding as tfe
    from paper_2607_07388_b200.engine import mine_ngrams
    L = 50_000
    buf = torch.full((tfe.tfe_mine_workspace_bytes(L, 3) + 1,), 0x5A, dtype=torch.uint8, device=DEV)
    for seed in range(3):
        tok = synth.make_corpus(30 + seed, L)
        e_pt, e_pl, e_pc, e_found, e_distinct, e_hist = orc.mine_ngrams(tok, synth.VOCAB, (2, 3, 4), min_count=2, cap=L)
        got = mine_ngrams(torch.from_numpy(tok).to(DEV), vocab=synth.VOCAB, orders=(2, 3, 4), min_count=2, cap=L,
                          workspace=buf[1:])
        assert got.n_found == e_found
        np.testing.assert_array_equal(got.distinct, e_distinct)
        np.testing.assert_array_equal(got.hist, e_hist)
        np.testing.assert_array_equal(got.phrase_tokens.cpu().numpy(), e_pt)
        np.testing.assert_array_equal(got.count.cpu().numpy().view(np.uint32), e_pc)


# ------------------------------------------------------------------ initial residency from the counts
def _assign_both(orc, count, G, hm):
    from paper_2607_07388_b200.engine import assign_residency
    e_slot, e_tiers = orc.assign_residency(count, G, hm)
    g_slot, g_tiers = assign_residency(torch.from_numpy(count.view(np.int32).copy()).to(DEV), G, hm)
    assert g_tiers == e_tiers
    np.testing.assert_array_equal(g_slot.cpu().numpy()[:len(count)], e_slot)
    return e_slot


@pytest.mark.parametrize("seed", range(int(os.environ.get("TFE_RANDOM_CASES", "24"))))
def test_assign_residency_random(orc, seed):
    rng = np.random.default_rng([6, seed])
    N = int(rng.choice([1, 2, 31, 1023, 1024, 1025, 5000, 70_000, 300_000]))
    kind = seed % 4
    if kind == 0:
        count = rng.integers(1, 4, size=N)                       # almost everything ties
    elif kind == 1:
        count = rng.zipf(1.5, size=N)                            # heavy tail
    elif kind == 2:
        count = rng.integers(0, 2**32, size=N, dtype=np.uint64)  # all 32 bits in use
    else:
        count = np.full(N, 7)                                    # one value
    count = np.minimum(count, 2**32 - 1).astype(np.uint32)
    for G in sorted({0, 1, N // 3, N - 1 if N > 1 else 1, N, N + 9}):
        _assign_both(orc, count, int(G), int(rng.integers(0, 5)))


def test_corpus_to_lookups_with_residency_from_counts(orc):
    """corpus -> phrase table -> residency from the counts -> index -> lookups, every step on the device, against
    the same chain run by the oracle on its own outputs."""
    import parity_harness as H
    from paper_2607_07388_b200.engine import Engram, assign_residency, bf16_tensor_from_bits, mine_ngrams
    L, orders, d = 200_000, (2, 3, 4), 32
    corpus = synth.make_corpus(41, L)
    got = mine_ngrams(torch.from_numpy(corpus).to(DEV), vocab=synth.VOCAB, orders=orders, min_count=2, cap=L)
    e_pt, e_pl, e_pc, e_found, _, _ = orc.mine_ngrams(corpus, synth.VOCAB, orders, min_count=2, cap=L)
    N = e_found
    C = N // 4
    e_slot, e_tiers = orc.assign_residency(e_pc, C, host_min_count=3)
    g_slot, g_tiers = assign_residency(got.count, C, host_min_count=3)
    assert g_tiers == e_tiers and e_tiers[0] == C and e_tiers[1] > 0 and e_tiers[2] > 0
    np.testing.assert_array_equal(g_slot.cpu().numpy(), e_slot)
    rows = synth.gaussian_bf16([41, 5], (C, d), 1 / 32)
    eng = Engram(got.phrase_tokens, got.phrase_len, g_slot, bf16_tensor_from_bits(rows, DEV), vocab=synth.VOCAB,
                 orders=orders, device_build=True)
    pr = H.Pair.__new__(H.Pair)
    pr.rows_bits, pr.d, pr.C, pr.orders, pr.hidden_dtype, pr.eng = rows, d, C, orders, 0, eng
    pr.ora = orc.Oracle(e_pt, e_pl, e_slot, rows.copy(), d=d, vocab=synth.VOCAB, orders=orders, gpu_slots=C)
    tok = corpus[50_000:50_000 + 4 * 512].reshape(4, 512).copy()
    h = synth.gaussian_bf16([41, 6], (4 * 512, d), 1.0)
    _, ref, info = pr.run_and_compare(tok, h, lam=1.0)
    assert info["n_hit"] > 300 and info["n_miss"] > 100
    assert set(np.unique(ref.miss_tier).tolist()) == {2, 3}                   # host and SSD entries both met
    pr.close()
