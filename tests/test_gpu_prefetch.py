"""GPU parity of tfe_prefetch_candidates (candidate expansion + priority, paper Sec. 4.4) against
the CPU oracle: phrase ids, tiers, sources and counts bit-exact; priorities bit-exact too, because
both sides form the product p*r*c in single precision in the same order and the ranking hangs on it."""
import os

import numpy as np
import pytest
import torch

from paper_2607_07388_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module")
def H():
    from paper_2607_07388_b200 import build
    build.build()
    from oracle import tfe_oracle
    tfe_oracle.build()
    import parity_harness
    return parity_harness


def _inputs(w, tb, B, K, seed, planted=0.5):
    """History of n_max-1 tokens per sequence + K predicted tokens; about `planted` of the
    (sequence, token) pairs continue a run of the table stream, the rest are filler."""
    rng = np.random.default_rng([w.seed, 21, seed])
    n_max = max(w.orders)
    Hh = n_max - 1
    cdf = synth.zipf_cdf(w.vocab, w.s)
    perm_query = np.random.default_rng([w.seed, 4]).permutation(w.vocab)
    hist = synth.zipf_tokens(rng, B * Hh, cdf, perm_query).reshape(B, Hh)
    cand = synth.zipf_tokens(rng, B * K, cdf, perm_query).reshape(B, K)
    src = rng.integers(0, tb.safe_len - n_max, size=B)
    seq_planted = rng.random(B) < 0.8
    for b in range(B):
        if seq_planted[b]:
            hist[b] = tb.stream[src[b]:src[b] + Hh]
            cand[b, 0] = tb.stream[src[b] + Hh]                 # the true continuation
            # other continuations of the same history that occur in the stream
            pos = np.nonzero(tb.stream[:tb.safe_len - 1] == hist[b, -1])[0][: int(planted * K)]
            for j, ppos in enumerate(pos[1:], start=1):
                if j < K:
                    cand[b, j] = tb.stream[ppos + 1]
    prob = rng.random((B, K)).astype(np.float32)
    prob /= prob.sum(axis=1, keepdims=True)
    prob[:, K // 2] = prob[:, 0]                                 # ties
    return hist.astype(np.int32), cand.astype(np.int32), prob.astype(np.float32)


def _compare(pr, hist, cand, prob, use, budget, c_host, c_ssd):
    t = lambda a: torch.from_numpy(a).to(DEV)
    ph, tr, sc, sr, cnt = pr.eng.prefetch_candidates(t(hist), t(cand), t(prob),
                                                     usefulness=None if use is None else t(use),
                                                     benefit_host=c_host, benefit_ssd=c_ssd, budget=budget)
    torch.cuda.synchronize()
    eph, etr, esc, esr, total = pr.ora.prefetch_candidates(hist, cand, prob, usefulness=use, benefit_host=c_host,
                                                           benefit_ssd=c_ssd, budget=budget)
    n = int(cnt[0].item())
    assert int(cnt[1].item()) == total and n == len(eph)
    np.testing.assert_array_equal(ph[:n].cpu().numpy().view(np.uint32), eph)
    assert (ph[n:budget].cpu().numpy().view(np.uint32) == 0xFFFFFFFF).all()      # the unused part of the budget: no phrase
    np.testing.assert_array_equal(tr[:n].cpu().numpy(), etr)
    np.testing.assert_array_equal(sr[:n].cpu().numpy().view(np.uint32), esr)
    np.testing.assert_array_equal(sc[:n].cpu().numpy().view(np.uint32), esc.view(np.uint32))
    return n, total


@pytest.mark.parametrize("orders,B,K", [((2, 3), 64, 16), ((2, 3, 4), 33, 64), ((1, 2), 5, 128), ((3,), 256, 8)])
def test_prefetch_candidates_match_the_oracle(H, orders, B, K):
    w = synth.config(2, n_phrases=200_000, gpu_slots=40_000, residency="hot_host_ssd", orders=orders, d=64,
                     rows="procedural")
    tb, pr = H.pair_from_workload(w)
    rng = np.random.default_rng(3)
    use = rng.choice([0.0, 0.5, 1.0, 1.0, 2.0, 3.5], size=w.n_phrases).astype(np.float32)
    totals = []
    for seed in range(3):
        hist, cand, prob = _inputs(w, tb, B, K, seed)
        for budget, u in ((4096, use), (7, use), (4096, None), (0, None)):
            n, total = _compare(pr, hist, cand, prob, u, budget, 1.0, 2.5)
            totals.append(total)
    assert max(totals) > 10
    # a benefit of zero for a tier removes its candidates; padding ids and short histories give none
    _compare(pr, hist, cand, prob, use, 100, 0.0, 1.0)
    cand_bad = cand.copy(); cand_bad[:, ::2] = -1; cand_bad[:, 1::4] = w.vocab
    _compare(pr, hist, cand_bad, prob, use, 4096, 1.0, 2.0)
    _compare(pr, hist[:, 1:] if hist.shape[1] > 1 else hist, cand, prob, use, 4096, 1.0, 2.0)
    pr.close()


def test_prefetch_budget_cut_with_many_candidates(H):
    # more candidates than the largest budget: the radix selection has to find the cut
    w = synth.config(2, n_phrases=300_000, gpu_slots=1_000, residency="hot_host_ssd", orders=(2, 3), d=64,
                     rows="procedural")
    tb, pr = H.pair_from_workload(w)
    B, K = 256, 128
    hist, cand, prob = _inputs(w, tb, B, K, 9, planted=1.0)
    prob[:] = np.float32(1.0 / K)                               # massive ties: order decided by the index
    n, total = _compare(pr, hist, cand, prob, None, 4096, 1.0, 1.0)
    assert total > 4096 and n == 4096
    n, total = _compare(pr, hist, cand, prob, None, 1000, 1.0, 3.0)
    pr.close()


@pytest.mark.parametrize("seed", range(int(os.environ.get("TFE_RANDOM_CASES", "16"))))
def test_prefetch_random_configurations(H, seed):
    """Seeded random orders, vocabulary, batch, top-K, history length, budget, benefits and usefulness."""
    rng = np.random.default_rng([515, seed])
    orders = tuple(o for o in (1, 2, 3, 4) if rng.random() < 0.6) or (2,)
    vocab = int(rng.choice([300, 4096, synth.VOCAB]))
    n_phrases = int(rng.integers(500, 60_000))
    n_phrases = min(n_phrases, sum(min(vocab ** n, 10 ** 6) for n in orders) // 4)      # what the tuple space allows
    w = synth.config(2, n_phrases=max(n_phrases, 16), gpu_slots=max(4, int(n_phrases * rng.uniform(0.05, 0.8))),
                     residency=str(rng.choice(["hot_host", "hot_host_ssd"])), orders=orders, d=16, rows="gaussian",
                     vocab=vocab)
    tb, pr = H.pair_from_workload(w, max_kicks=100_000)
    B, K = int(rng.integers(1, 300)), int(rng.integers(1, 129))
    if max(orders) == 1:                     # single tokens are the phrases: no history at all
        hist = np.zeros((B, 0), np.int32)
        cand = rng.choice(tb.stream[:tb.safe_len], size=(B, K)).astype(np.int32)
        cand[:, ::3] = rng.integers(0, vocab, size=cand[:, ::3].shape)
        prob = rng.random((B, K)).astype(np.float32)
    else:
        hist, cand, prob = _inputs(w, tb, B, K, seed, planted=float(rng.uniform(0.2, 1.0)))
    if rng.random() < 0.3 and hist.shape[1] > 1:
        hist = np.ascontiguousarray(hist[:, 1:])                # a history shorter than the longest order needs
    if rng.random() < 0.3:
        prob[:] = np.float32(0.25)                               # ties everywhere
    use = None if rng.random() < 0.4 else rng.choice([0.0, 0.5, 1.0, 2.0], size=w.n_phrases).astype(np.float32)
    budget = int(rng.choice([0, 1, 13, 256, 4096]))
    c_host, c_ssd = float(rng.choice([0.0, 1.0, 1.5])), float(rng.choice([0.0, 2.0, 3.0]))
    if hist.shape[1] == 0:
        hist = np.zeros((B, 0), np.int32)
    _compare(pr, hist, cand, prob, use, budget, c_host, c_ssd)
    pr.close()
