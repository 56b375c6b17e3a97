"""tfe_cache_install_device: batches that live on the device and were never checked by the host,
against the oracle's lenient installation; and the prefetch loop without a host round trip."""
import os

import numpy as np
import pytest
import torch

from paper_2607_07388_b200 import synth

pytestmark = pytest.mark.gpu
DEV = torch.device("cuda:0")


@pytest.fixture(scope="module")
def H():
    import parity_harness
    return parity_harness


def _to_dev(a, dtype):
    return torch.from_numpy(np.ascontiguousarray(a)).to(DEV, dtype)


def _install_both(pr, w, ids, dst):
    """One batch on both sides; src row k is the phrase's own row (any content for ids that are no phrases)."""
    safe = np.minimum(ids.astype(np.int64), w.n_phrases - 1)
    src = synth.phrase_rows_np(w, safe)
    e_applied, e_cnt = pr.ora.cache_install_lenient(ids, src, dst)
    from paper_2607_07388_b200.engine import bf16_tensor_from_bits
    g_applied, g_cnt = pr.eng.cache_install_device(_to_dev(ids.view(np.int32), torch.int32), bf16_tensor_from_bits(src, DEV),
                                                   _to_dev(dst, torch.int32))
    torch.cuda.synchronize()
    np.testing.assert_array_equal(g_applied.cpu().numpy(), e_applied)
    assert int(g_cnt.item()) == e_cnt
    return e_applied, e_cnt


@pytest.mark.parametrize("seed", range(int(os.environ.get("TFE_RANDOM_CASES", "12"))))
def test_device_install_random_batches(H, seed):
    rng = np.random.default_rng([1313, seed])
    n_phrases = int(rng.integers(300, 20_000))
    gpu_slots = max(16, int(n_phrases * rng.uniform(0.1, 0.8)))
    w = synth.config(1, B=3, T=int(rng.integers(60, 300)), n_phrases=n_phrases, gpu_slots=gpu_slots, d=int(rng.choice([16, 64, 256])),
                     residency="hot_host_ssd", reserve_free=int(gpu_slots * rng.uniform(0, 0.3)), p=0.5,
                     orders=(2, 3) if rng.random() < 0.5 else (2, 3, 4))
    tb, pr = H.pair_from_workload(w, device_build=bool(rng.random() < 0.5))
    if rng.random() < 0.5:
        pr.eng.cache_policy_enable()
        policy_on = True
    else:
        policy_on = False
    h = synth.make_hidden_np(w)
    total_applied = 0
    for step in range(int(rng.integers(2, 6))):
        tok = synth.make_queries(w, tb, variant=step % 3)
        _, ref, _ = pr.run_and_compare(tok, h, lam=1.0)
        if policy_on:
            pr.ora.touch(ref)
        n = int(rng.integers(1, 600))
        # a mix: missed phrases, resident phrases, ids that are no phrases, repeats; slots: free, occupied,
        # out of range, repeats
        pool = np.concatenate([ref.miss_phrase.astype(np.int64), rng.integers(0, n_phrases + 50, size=n)])
        ids = rng.choice(pool, size=n).astype(np.uint32)
        dst = rng.integers(-2, gpu_slots + 3, size=n).astype(np.int32)
        if rng.random() < 0.5:
            dst[: n // 2] = rng.permutation(gpu_slots)[: n // 2] if gpu_slots >= n // 2 else dst[: n // 2]
        applied, cnt = _install_both(pr, w, ids, dst)
        total_applied += cnt
        pr.run_and_compare(tok, h, lam=1.0)                      # the new residency state answers like the oracle's
        if policy_on:
            pr.ora.touch(pr.ora.lookup(tok))
            freq, last, epoch = pr.eng.cache_stats()
            assert epoch == pr.ora.epoch
            np.testing.assert_array_equal(freq, pr.ora.freq)
            np.testing.assert_array_equal(last, pr.ora.last)
    assert total_applied > 0
    # the host-side installation still works afterwards (its residency copy is refreshed from the device)
    from paper_2607_07388_b200 import binding as tfe
    res = pr.ora.lookup(tok)
    want = np.unique(res.miss_phrase)[:5].astype(np.uint32)
    if len(want):
        free = np.arange(len(want), dtype=np.int32)
        src = synth.phrase_rows_np(w, want)
        assert pr.ora.cache_install(want, src, free) == 0
        pr.eng.cache_install(want, src, free)
        pr.run_and_compare(tok, h, lam=1.0)
        with pytest.raises(tfe.TfeError) as e:
            pr.eng.cache_install(want[:1], src[:1], free[:1])
        assert e.value.status == tfe.TFE_ERR_ALREADY_RESIDENT
    pr.close()


def test_device_install_argument_checks_and_empty_batch(H):
    from paper_2607_07388_b200 import binding as tfe
    w = synth.config(1)
    tb, pr = H.pair_from_workload(w)
    ids = torch.zeros(4, dtype=torch.int32, device=DEV); dst = torch.zeros(4, dtype=torch.int32, device=DEV)
    rows = torch.zeros((4, w.d), dtype=torch.bfloat16, device=DEV)
    cnt = torch.full((1,), 7, dtype=torch.int32, device=DEV)
    tfe.tfe_cache_install_device(pr.eng.ctx, 0, ids, rows, dst, None, cnt)
    assert int(cnt.item()) == 0
    for n in (-1, tfe.INSTALL_DEVICE_MAX + 1):
        with pytest.raises(tfe.TfeError):
            tfe.tfe_cache_install_device(pr.eng.ctx, n, ids, rows, dst)
    with pytest.raises(tfe.TfeError):
        tfe.tfe_cache_install_device(pr.eng.ctx, 4, None, rows, dst)
    pr.close()


def test_prefetch_loop_without_a_host_round_trip(H):
    """Head -> candidates -> victims -> rows gathered on the device -> installation: every step takes the
    previous step's DEVICE output and nothing is copied to the host in between.  The oracle runs the same
    chain with its own functions on its own outputs; afterwards both hold the same state (slot by slot).
    The head's probabilities are put on a grid of 1/64 on both sides (the caller's choice of how to weigh
    them), so that the two priority orders are the same numbers and not two roundings of near-equal ones."""
    from oracle import tfe_oracle as orc
    from paper_2607_07388_b200 import binding as tfe
    from paper_2607_07388_b200.engine import EarlyExitHead, bf16_tensor_from_bits, _device_view
    w = synth.config(2, B=24, n_phrases=40_000, gpu_slots=5_000, d=64)
    tb, pr = H.pair_from_workload(w)
    pr.eng.cache_policy_enable()
    B, V, dh, K, budget = w.B, w.vocab, 64, 8, 256
    rng = np.random.default_rng(29)
    Wf = rng.integers(-2, 3, size=(V, dh)).astype(np.float32)
    W_bits = synth.f32_to_bf16_bits(Wf)
    head = EarlyExitHead(bf16_tensor_from_bits(W_bits, DEV), max_batch=B)
    all_rows_np = synth.phrase_rows_np(w, np.arange(w.n_phrases))
    all_rows = bf16_tensor_from_bits(all_rows_np, DEV)              # the fetched rows, staged on the device
    pos = tb.safe_len - 40 * B + 40 * np.arange(B)
    hid = synth.make_hidden_np(w, Q=B)
    installed = 0
    for step in range(5):
        tok = np.stack([tb.stream[p - 2:p + 1] for p in pos]).astype(np.int32)
        _, ref, _ = pr.run_and_compare(tok, hid, q_start=2, lam=1.0)
        pr.ora.touch(ref)
        nxt = tb.stream[pos + 1]
        hf = np.stack([np.sign(Wf[t]) + (Wf[t] == 0) for t in nxt]).astype(np.float32)
        h_bits = synth.f32_to_bf16_bits(hf)
        # ---- the device chain
        t_tok, t_prob = head.topk(bf16_tensor_from_bits(h_bits, DEV), K)
        t_prob = torch.round(t_prob * 64) / 64
        hist = torch.from_numpy(np.ascontiguousarray(tok[:, 1:])).to(DEV)
        ph = torch.full((budget,), -1, dtype=torch.int32, device=DEV)                 # unwritten entries are no phrases
        tr = torch.empty(budget, dtype=torch.uint8, device=DEV); sc = torch.empty(budget, dtype=torch.float32, device=DEV)
        sr = torch.empty(budget, dtype=torch.int32, device=DEV); cnt = torch.zeros(2, dtype=torch.int32, device=DEV)
        tfe.tfe_prefetch_candidates(pr.eng.ctx, hist, B, 2, t_tok, t_prob, K, out_phrase=ph, out_tier=tr, out_score=sc,
                                    out_src=sr, out_count=cnt, budget=budget, benefit_host=1.0, benefit_ssd=2.0)
        assert tfe.tfe_cache_select_victims_async(pr.eng.ctx, budget, half_life=2) == budget
        slots_ptr, _ = tfe.tfe_cache_select_victims_device(pr.eng.ctx)
        slots_dev = _device_view(slots_ptr, (budget,), "<i4", DEV)
        src = all_rows[ph.clamp(0, w.n_phrases - 1).long()]                            # gather on the device
        applied, n_applied = pr.eng.cache_install_device(ph, src, slots_dev)
        # ---- the oracle's chain, on its own outputs
        e_tok, e_prob, _ = orc.head_topk(orc.head_logits(W_bits, h_bits), K)
        e_prob = (np.round(e_prob * 64) / 64).astype(np.float32)
        eph, etr, esc, esr, total = pr.ora.prefetch_candidates(tok[:, 1:], e_tok, e_prob, benefit_host=1.0, benefit_ssd=2.0,
                                                               budget=budget)
        e_slots, _ = pr.ora.cache_victims(budget, half_life=2)
        ids_full = np.full(budget, 0xFFFFFFFF, np.uint32); ids_full[:len(eph)] = eph
        e_applied, e_cnt = pr.ora.cache_install_lenient(ids_full, all_rows_np[np.minimum(ids_full, w.n_phrases - 1)], e_slots)
        # ---- now compare
        torch.cuda.synchronize()
        np.testing.assert_array_equal(t_tok.cpu().numpy(), e_tok)
        np.testing.assert_array_equal(t_prob.cpu().numpy(), e_prob)
        np.testing.assert_array_equal(ph.cpu().numpy().view(np.uint32), ids_full)
        np.testing.assert_array_equal(slots_dev.cpu().numpy(), e_slots)
        np.testing.assert_array_equal(applied.cpu().numpy(), e_applied)
        assert int(n_applied.item()) == e_cnt == min(total, budget)
        freq, last, epoch = pr.eng.cache_stats()
        assert epoch == pr.ora.epoch
        np.testing.assert_array_equal(freq, pr.ora.freq)
        np.testing.assert_array_equal(last, pr.ora.last)
        installed += e_cnt
        pos = pos + 1
    assert installed > 50
    tok = np.stack([tb.stream[p - 2:p + 1] for p in pos]).astype(np.int32)
    pr.run_and_compare(tok, hid, q_start=2, lam=1.0)
    head.close()
    pr.close()


def test_device_install_replayed_from_a_graph(H):
    """Victim selection + device-side installation captured once and replayed with new batches written into the
    same buffers: the call keeps no state on the host, so every replay must act like a fresh call."""
    from paper_2607_07388_b200 import binding as tfe
    from paper_2607_07388_b200.engine import bf16_tensor_from_bits, _device_view
    w = synth.config(1, B=3, T=128, n_phrases=6_000, gpu_slots=1_500, d=64, residency="hot_host_ssd", p=0.5)
    tb, pr = H.pair_from_workload(w)
    pr.eng.cache_policy_enable()
    n = 64
    ids_buf = torch.zeros(n, dtype=torch.int32, device=DEV)
    src_buf = torch.zeros((n, w.d), dtype=torch.bfloat16, device=DEV)
    applied = torch.zeros(n, dtype=torch.uint8, device=DEV)
    cnt = torch.zeros(1, dtype=torch.int32, device=DEV)
    # first calls outside the capture (allocations), checked like any other
    tfe.tfe_cache_select_victims_async(pr.eng.ctx, n, 2)
    slots_ptr, _ = tfe.tfe_cache_select_victims_device(pr.eng.ctx)
    slots_dev = _device_view(slots_ptr, (n,), "<i4", DEV)
    pr.eng.cache_install_device(ids_buf.fill_(-1), src_buf, slots_dev)             # nothing valid: applies nothing
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            tfe.tfe_cache_select_victims_async(pr.eng.ctx, n, 2, stream=side)
            tfe.tfe_cache_install_device(pr.eng.ctx, n, ids_buf, src_buf, slots_dev, applied, cnt, stream=side)
    torch.cuda.synchronize()
    rng = np.random.default_rng(8)
    h = synth.make_hidden_np(w)
    total = 0
    for step in range(6):
        tok = synth.make_queries(w, tb, variant=step)
        _, ref, _ = pr.run_and_compare(tok, h, lam=1.0)
        pr.ora.touch(ref)
        # a batch with repeats of earlier steps' ids (now resident), invalid ids and fresh misses
        pool = np.concatenate([ref.miss_phrase.astype(np.int64), rng.integers(0, w.n_phrases + 20, size=n)])
        ids = rng.choice(pool, size=n).astype(np.uint32)
        src = synth.phrase_rows_np(w, np.minimum(ids.astype(np.int64), w.n_phrases - 1))
        ids_buf.copy_(torch.from_numpy(ids.view(np.int32)))
        src_buf.copy_(bf16_tensor_from_bits(src, DEV))
        graph.replay()
        torch.cuda.synchronize()
        e_slots, _ = pr.ora.cache_victims(n, 2)
        e_applied, e_cnt = pr.ora.cache_install_lenient(ids, src, e_slots)
        np.testing.assert_array_equal(slots_dev.cpu().numpy(), e_slots)
        np.testing.assert_array_equal(applied.cpu().numpy(), e_applied)
        assert int(cnt.item()) == e_cnt
        total += e_cnt
        pr.run_and_compare(tok, h, lam=1.0)
        pr.ora.touch(pr.ora.lookup(tok))
    assert total > 30
    pr.close()
