"""GPU-tier retention ranking (frequency / recency bookkeeping in the lookup kernels, victim
selection) against the oracle's state machine, through the C ABI."""
import os

import numpy as np
import pytest
import torch

from paper_2607_07388_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def H():
    import parity_harness
    return parity_harness


def _compare_state(pr):
    freq, last, epoch = pr.eng.cache_stats()
    assert epoch == pr.ora.epoch
    np.testing.assert_array_equal(freq, pr.ora.freq)
    np.testing.assert_array_equal(last, pr.ora.last)


def _compare_victims(pr, n, half_life):
    slots, keys = pr.eng.cache_select_victims(n, half_life)
    e_slots, e_keys = pr.ora.cache_victims(n, half_life)
    np.testing.assert_array_equal(slots, e_slots)
    np.testing.assert_array_equal(keys, e_keys)
    return e_slots          # the oracle's own (equal) values: nothing the GPU computed feeds the oracle


@pytest.mark.parametrize("policy", [0, 1])
def test_bookkeeping_and_victims_follow_the_oracle(H, policy):
    w = synth.config(1, B=6, T=300, n_phrases=30_000, gpu_slots=9_000, residency="hot_host", p=0.7,
                     reserve_free=500)
    tb, pr = H.pair_from_workload(w)
    pr.eng.cache_policy_enable()
    h = synth.make_hidden_np(w)
    for step in range(5):
        tok = synth.make_queries(w, tb, variant=step % 3)      # repeats make some slots hotter
        g, ref, _ = pr.run_and_compare(tok, h, policy=policy, lam=1.0)
        pr.ora.touch(ref)
        _compare_state(pr)
    assert pr.ora.freq.max() >= 3 and (pr.ora.freq > 0).sum() > 300
    for n, hl in ((1, 0), (37, 0), (500, 0), (501, 1), (2000, 2), (4096, 0), (4096, 3)):
        _compare_victims(pr, n, hl)
    # install over the 64 worst slots (all free here), then over 64 occupied ones; state and ranking follow
    res = pr.ora.lookup(tok, policy=policy)
    want = np.unique(res.miss_phrase)[:128].astype(np.uint32)
    assert len(want) == 128
    for part in (want[:64], want[64:]):
        if part is want[64:]:
            dst = _compare_victims(pr, 700, 2)[-64:].copy()         # occupied, least worth keeping after the free ones
            assert (pr.ora.slot_owner[dst] >= 0).all()
        else:
            dst = _compare_victims(pr, 64, 2).copy()
            assert (pr.ora.slot_owner[dst] < 0).all()
        src = synth.phrase_rows_np(w, part)
        assert pr.ora.cache_install(part, src, dst) == 0
        pr.eng.cache_install(part, src, dst)
        _compare_state(pr)
        g, ref, _ = pr.run_and_compare(tok, h, policy=policy, lam=1.0)
        pr.ora.touch(ref)
        _compare_state(pr)
        _compare_victims(pr, 1000, 2)
    pr.close()


# (list_cap, final_cap, n_samples): every path of the selection on one history -- the whole table in the list;
# a sampled threshold with and without refine steps; a list that overflows (the table is walked again); a
# threshold from a single sample (mostly too low: the table is walked again); the defaults
_TUNINGS = [(0, 0, 0), (16384, 4500, 0), (1024, 0, 256), (1024, 4200, 64), (64, 0, 2048), (8192, 4500, 1), (300, 4100, 7),
            (2000, 1, 2048)]


@pytest.mark.parametrize("ties", [False, True])
def test_selection_result_is_independent_of_its_internal_sizes(H, ties):
    from paper_2607_07388_b200 import binding as tfe
    w = synth.config(1, B=6, T=300, n_phrases=40_000, gpu_slots=13_001, residency="hot_host", p=0.7,
                     reserve_free=0 if ties else 700)
    tb, pr = H.pair_from_workload(w)
    pr.eng.cache_policy_enable()
    h = synth.make_hidden_np(w)
    for step in range(0 if ties else 6):       # ties: nothing looked up, every key equal, the slot decides
        tok = synth.make_queries(w, tb, variant=step % 3)
        g, ref, _ = pr.run_and_compare(tok, h, lam=1.0)
        pr.ora.touch(ref)
    with pytest.raises(tfe.TfeError):
        tfe.tfe_cache_select_tuning(pr.eng.ctx, 1_048_577, 0, 0)
    for list_cap, final_cap, n_samples in _TUNINGS:
        tfe.tfe_cache_select_tuning(pr.eng.ctx, list_cap, final_cap, n_samples)
        for n, hl in ((1, 0), (33, 1), (700, 2), (701, 0), (4096, 3), (4095, 0)):
            _compare_victims(pr, n, hl)
    pr.close()


def test_policy_off_and_argument_checks(H):
    from paper_2607_07388_b200 import binding as tfe
    w = synth.config(1)
    tb, pr = H.pair_from_workload(w)
    with pytest.raises(tfe.TfeError):
        pr.eng.cache_select_victims(4)             # bookkeeping not enabled
    pr.eng.cache_policy_enable()
    with pytest.raises(tfe.TfeError):
        pr.eng.cache_select_victims(tfe.VICTIMS_MAX + 1)
    with pytest.raises(tfe.TfeError):
        pr.eng.cache_select_victims(4, half_life=1 << 26)      # 32 half-lives must stay below 2^31 epochs
    slots, keys = pr.eng.cache_select_victims(3, half_life=(1 << 26) - 1)
    np.testing.assert_array_equal(slots, np.arange(3))
    slots, keys = pr.eng.cache_select_victims(0)
    assert len(slots) == 0
    # nothing looked up yet: every owned slot has freq 0, age 0 -> key 65535, ascending slot order
    slots, keys = pr.eng.cache_select_victims(100)
    np.testing.assert_array_equal(slots, np.arange(100))
    assert (keys == 65535).all()
    # enabling again clears the state
    tok = synth.make_queries(w, tb)
    g, ref, _ = pr.run_and_compare(tok, synth.make_hidden_np(w), lam=1.0)
    assert pr.eng.cache_stats()[2] == 1
    pr.eng.cache_policy_enable()
    freq, last, epoch = pr.eng.cache_stats()
    assert epoch == 0 and freq.sum() == 0 and last.sum() == 0
    pr.close()


def test_victims_more_than_slots_and_host_pipeline_epoch(H):
    # fewer slots than requested: all of them come back, ranked; the piecewise host-buffer call
    # counts as one lookup (one epoch) and bumps every injected slot once per hit
    from paper_2607_07388_b200 import binding as tfe
    w = synth.config(1, B=6, T=2731, d=1024, n_phrases=3_000, gpu_slots=1_500, residency="hot_host", p=0.6)
    tb, pr = H.pair_from_workload(w)
    pr.eng.cache_policy_enable()
    tok = synth.make_queries(w, tb)
    h = synth.make_hidden_np(w)
    out = np.empty_like(h)
    tfe.tfe_lookup_inject_host(pr.eng.ctx, tok, w.B, w.T, 0, h, out, lam=1.0)
    torch.cuda.synchronize()
    ref = pr.ora.lookup(tok)
    pr.ora.touch(ref)
    _compare_state(pr)
    slots = _compare_victims(pr, 4096, 0)
    assert len(slots) == 1500 and len(set(slots.tolist())) == 1500
    pr.close()


@pytest.mark.parametrize("seed", range(int(os.environ.get("TFE_RANDOM_CASES", "10"))))
def test_policy_random_histories(H, seed):
    """Seeded random interleavings of lookups (either policy), victim selections (any n, any half-life)
    and installs into the selected victims: bookkeeping and ranking follow the oracle at every step."""
    from paper_2607_07388_b200 import binding as tfe
    rng = np.random.default_rng([808, seed])
    n_phrases = int(rng.integers(200, 20_000))
    gpu_slots = max(8, int(n_phrases * rng.uniform(0.1, 0.9)))
    w = synth.config(1, B=int(rng.integers(1, 6)), T=int(rng.integers(40, 300)), n_phrases=n_phrases, gpu_slots=gpu_slots,
                     residency="hot_host_ssd", reserve_free=int(gpu_slots * rng.uniform(0.0, 0.3)), p=0.5,
                     orders=(2, 3) if rng.random() < 0.5 else (2, 3, 4), d=16)
    tb, pr = H.pair_from_workload(w, device_build=bool(rng.random() < 0.5))
    pr.eng.cache_policy_enable()
    h = synth.make_hidden_np(w)
    for step in range(int(rng.integers(3, 9))):
        tok = synth.make_queries(w, tb, variant=int(rng.integers(0, 3)))
        policy = int(rng.random() < 0.4)
        _, ref, _ = pr.run_and_compare(tok, h, policy=policy, lam=1.0)
        pr.ora.touch(ref)
        _compare_state(pr)
        n = int(rng.choice([1, 5, 64, 1000, 4096]))
        hl = int(rng.choice([0, 1, 2, 5]))
        # the sizes of the selection's internal steps never change its result
        tfe.tfe_cache_select_tuning(pr.eng.ctx, int(rng.choice([0, 16, 200, 3000])), int(rng.choice([0, 2, 700, 4500])),
                                    int(rng.choice([0, 1, 9, 300, 2048])))
        slots = _compare_victims(pr, n, hl)
        if rng.random() < 0.7:
            want = np.unique(pr.ora.lookup(tok, policy=policy).miss_phrase).astype(np.uint32)
            k = int(min(len(want), len(slots), rng.integers(1, 200)))
            if k:
                src = synth.phrase_rows_np(w, want[:k])
                assert pr.ora.cache_install(want[:k], src, slots[:k].copy()) == 0
                pr.eng.cache_install(want[:k], src, slots[:k].copy())
                _compare_state(pr)
    pr.close()
