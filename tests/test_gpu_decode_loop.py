"""The decode loop of Sec. 4.3 / 4.4 end to end on the device, every step against the oracle:
lookup-and-inject on the current tokens, early-exit head on the hidden states, candidate phrases of
the predicted tokens with their priorities, victims from the retention ranking, installation of the
fetched rows -- and then the next tokens arrive and the prefetched phrases are hits."""
import numpy as np
import pytest
import torch

from paper_2607_07388_b200 import synth

pytestmark = pytest.mark.gpu
DEV = torch.device("cuda:0")


def test_prefetch_loop_turns_predicted_misses_into_hits():
    import parity_harness as H
    from oracle import tfe_oracle as orc
    from paper_2607_07388_b200.engine import EarlyExitHead, bf16_tensor_from_bits
    w = synth.config(2, B=32, n_phrases=50_000, gpu_slots=6_000, d=256)
    tb, pr = H.pair_from_workload(w)
    pr.eng.cache_policy_enable()
    B, V, dh, K = w.B, w.vocab, 64, 8
    rng = np.random.default_rng(23)
    # sequences follow the table stream from late positions (rare phrases, mostly outside the GPU tier)
    pos = tb.safe_len - 40 * B + 40 * np.arange(B)
    # the head: small-integer weights (exact fp32 logits); the hidden state of sequence b at a step points
    # at the row of its true next token, so that token is predicted first
    Wf = rng.integers(-2, 3, size=(V, dh)).astype(np.float32)
    W_bits = synth.f32_to_bf16_bits(Wf)
    head = EarlyExitHead(bf16_tensor_from_bits(W_bits, DEV), max_batch=B)
    hid_main = synth.make_hidden_np(w, Q=B)
    hits_with, hits_without = 0, 0
    shadow = orc.Oracle(tb.phrase_tokens, tb.phrase_len, tb.init_slot, pr.rows_bits.copy(), d=w.d, vocab=w.vocab,
                        orders=w.orders, gpu_slots=pr.C)           # the same table with no prefetching at all
    for step in range(6):
        tok = np.stack([tb.stream[p - 2:p + 1] for p in pos]).astype(np.int32)          # [B, 3], query at the last
        # 1. lookup and inject, bookkeeping
        _, ref, _ = pr.run_and_compare(tok, hid_main, q_start=2, lam=1.0)
        pr.ora.touch(ref)
        freq, last, epoch = pr.eng.cache_stats()
        assert epoch == pr.ora.epoch and np.array_equal(freq, pr.ora.freq) and np.array_equal(last, pr.ora.last)
        hits_with += int((ref.flags == 1).sum())
        hits_without += int((shadow.lookup(tok, 2).flags == 1).sum())
        # 2. early-exit head: the next token of the stream gets the largest logit
        nxt = tb.stream[pos + 1]
        hf = np.zeros((B, dh), np.float32)
        for b in range(B):
            hf[b] = np.sign(Wf[nxt[b]]) + (Wf[nxt[b]] == 0)
        h_bits = synth.f32_to_bf16_bits(hf)
        t_tok, t_prob = head.topk(bf16_tensor_from_bits(h_bits, DEV), K)
        assert head.status() == 0
        e_tok, e_prob, _ = orc.head_topk(orc.head_logits(W_bits, h_bits), K)
        np.testing.assert_array_equal(t_tok.cpu().numpy(), e_tok)
        assert (e_tok[:, 0] == nxt).mean() > 0.9
        # 3. candidate phrases of the predicted tokens, by priority
        hist = torch.from_numpy(np.ascontiguousarray(tok[:, 1:])).to(DEV)               # the last two tokens
        ph, tr, sc, sr, cnt = pr.eng.prefetch_candidates(hist, t_tok, t_prob, benefit_host=1.0, benefit_ssd=2.0, budget=4096)
        torch.cuda.synchronize()
        # the oracle's chain runs on the oracle head's own outputs (nothing the GPU computed goes into it)
        eph, etr, esc, esr, total = pr.ora.prefetch_candidates(tok[:, 1:], e_tok, e_prob.astype(np.float32),
                                                               benefit_host=1.0, benefit_ssd=2.0, budget=4096)
        n = int(cnt[0].item())
        assert n == len(eph) and int(cnt[1].item()) == total and total <= 4096
        got = sorted(zip(sr[:n].cpu().numpy().view(np.uint32).tolist(), ph[:n].cpu().numpy().view(np.uint32).tolist(),
                         tr[:n].cpu().numpy().tolist()))
        assert got == sorted(zip(esr.tolist(), eph.tolist(), etr.tolist()))
        np.testing.assert_allclose(np.sort(sc[:n].cpu().numpy()), np.sort(esc), rtol=1e-4)
        # 4. fetch: the distinct candidate phrases, best first; victims from the retention ranking
        ids = np.array(list(dict.fromkeys(eph.tolist())), np.uint32)
        if len(ids):
            g_slots, g_keys = pr.eng.cache_select_victims(len(ids), half_life=2)
            e_slots, e_keys = pr.ora.cache_victims(len(ids), half_life=2)
            np.testing.assert_array_equal(g_slots, e_slots)
            np.testing.assert_array_equal(g_keys, e_keys)
            # 5. install on both sides
            src = synth.phrase_rows_np(w, ids)
            assert pr.ora.cache_install(ids, src, e_slots) == 0
            pr.eng.cache_install(ids, src, g_slots)
        pos = pos + 1
    # the prefetched phrases were there when their tokens arrived
    print(f"GPU-tier hits over 6 steps of {B} sequences: {hits_with} with the prefetch loop, {hits_without} without")
    assert hits_with > hits_without + B, (hits_with, hits_without)
    head.close()
    pr.close()


def test_launch_overlap_respects_the_producer_on_the_stream():
    """The lookup is launched so that its set-up overlaps the kernel before it on the stream; it must still see
    everything that kernel wrote.  Producer -> lookup -> lookup chains with no host synchronisation in between:
    hidden states and ids written by torch kernels immediately before, and a lookup in place on the output of
    the previous one (the residual stream through two injection layers)."""
    import parity_harness as H
    w = synth.config(1, B=8, T=256, n_phrases=30_000, gpu_slots=30_000, d=512, p=0.5)
    tb, pr = H.pair_from_workload(w)
    rng = np.random.default_rng(77)
    for rep in range(20):
        tok = synth.make_queries(w, tb, variant=rep)
        h_np = synth.gaussian_bf16([77, rep], (w.Q, w.d), 1.0)
        # producers: ids arrive shifted and are fixed up on the device; h is the sum of two halves
        tok_shift = torch.from_numpy(tok + 5).to(H.DEV)
        h_full = H.bf16_tensor_from_bits(h_np, H.DEV)
        half = (h_full.float() * 0.5).to(torch.bfloat16)                      # exact: a power of two
        big = torch.empty(1 << 22, device=H.DEV)                              # keeps the stream busy before the producers
        torch.cuda.synchronize()
        big.normal_()
        tok_dev = tok_shift - 5                                               # producer kernel 1
        h_dev = half + half                                                   # producer kernel 2, directly before the lookup
        out1 = pr.eng.lookup_inject(tok_dev, h_dev, lam=1.0).out              # layer 1, out of place
        out2 = pr.eng.lookup_inject(tok_dev, out1, out1, lam=0.5).out         # layer 2, in place on layer 1's output
        torch.cuda.synchronize()
        ref = pr.ora.lookup(tok)
        _, r1 = pr.ora.inject(ref, h_np, lam=1.0)
        _, r2 = pr.ora.inject(ref, r1, lam=0.5)
        np.testing.assert_array_equal(H.bits_from_bf16_tensor(out2), r2)
    pr.close()
