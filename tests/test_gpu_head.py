"""Early-exit prefetch head (tcgen05 GEMM + softmax + top-K) against the fp64 oracle, through the C ABI."""
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


def _bits_to_gpu(bits):
    from paper_2607_07388_b200.engine import bf16_tensor_from_bits
    return bf16_tensor_from_bits(bits, DEV)


def _inputs(seed, V, d, B, w_scale=0.25):
    rng = np.random.default_rng(seed)
    W = synth.f32_to_bf16_bits((rng.standard_normal((V, d)) * w_scale).astype(np.float32))
    h = synth.f32_to_bf16_bits(rng.standard_normal((B, d)).astype(np.float32))
    return W, h


def check_topk(z64, tokens, prob, K, logit_tol, lse=None):
    """The K tokens returned for every row must be a valid top-K of the oracle's logits up to
    `logit_tol` (rows of W whose logits are closer than that may swap), carry the oracle's
    probabilities, and come in descending order."""
    B, V = z64.shape
    m = z64.max(axis=1, keepdims=True)
    lse64 = (m + np.log(np.exp(z64 - m).sum(axis=1, keepdims=True)))[:, 0]
    if lse is not None:
        np.testing.assert_allclose(lse, lse64, rtol=0, atol=5e-4)
    for b in range(B):
        t = tokens[b]
        assert len(set(t.tolist())) == K and t.min() >= 0 and t.max() < V
        kth = np.partition(z64[b], V - K)[V - K]                 # K-th largest oracle logit
        assert z64[b, t].min() >= kth - logit_tol, (b, z64[b, t].min(), kth)
        rest = np.ones(V, bool); rest[t] = False
        assert K == V or z64[b, rest].max() <= z64[b, t].min() + logit_tol
        p64 = np.exp(z64[b, t] - lse64[b])
        np.testing.assert_allclose(prob[b], p64, rtol=2e-3, atol=1e-9)
        assert (np.diff(prob[b]) <= 1e-7 * prob[b][:-1] + 1e-12).all()      # descending
        # clear winners (further than the tolerance from the cut) must be present, in the oracle's order
        order = np.argsort(-z64[b], kind="stable")
        clear = [v for v in order[:K] if z64[b, v] > kth + 2 * logit_tol]
        assert set(clear) <= set(t.tolist())


@pytest.mark.parametrize("V,d,B,K", [(1000, 64, 3, 16), (4096 + 72, 128, 17, 64), (20_000, 256, 64, 128),
                                     (148 * 128 * 2, 192, 33, 16), (333, 64, 1, 1), (50_000, 1024, 130, 64)])
def test_head_against_oracle(orc, V, d, B, K):
    from paper_2607_07388_b200.engine import EarlyExitHead
    W, h = _inputs(V + d + B, V, d, B)
    head = EarlyExitHead(_bits_to_gpu(W), max_batch=max(B, 16))
    tok, prob = head.topk(_bits_to_gpu(h), K)
    assert head.status() == 0
    z = head.logits(B).cpu().numpy()
    z64 = orc.head_logits(W, h)
    # bf16 products are exact in fp32; the error is the fp32 accumulation over d terms
    tol = 4e-6 * d * np.abs(z64).max()
    np.testing.assert_allclose(z, z64, rtol=0, atol=tol)
    check_topk(z64, tok.cpu().numpy(), prob.cpu().numpy(), K, logit_tol=2 * tol, lse=head.lse(B).cpu().numpy())
    # a second call with another batch on the same head (buffers and barriers are re-armed)
    W2, h2 = _inputs(V + 1, 8, d, min(B, 5))
    tok2, prob2 = head.topk(_bits_to_gpu(h2), min(K, 8))
    assert head.status() == 0
    z64b = orc.head_logits(W, h2)
    check_topk(z64b, tok2.cpu().numpy(), prob2.cpu().numpy(), min(K, 8), logit_tol=2 * tol)
    head.close()


def test_head_exact_cases(orc):
    """Logits that fp32 accumulates exactly: ties resolve by token id, probabilities are exact softmax."""
    from paper_2607_07388_b200.engine import EarlyExitHead
    V, d, B = 2000, 64, 4
    rng = np.random.default_rng(9)
    Wf = rng.integers(-4, 5, size=(V, d)).astype(np.float32)          # small integers: every partial sum is exact
    Wf[700] = Wf[20]; Wf[1500] = Wf[20]                                # three identical rows
    hf = rng.integers(-3, 4, size=(B, d)).astype(np.float32)
    hf[3] = 0                                                          # a zero state: uniform distribution
    W, h = synth.f32_to_bf16_bits(Wf), synth.f32_to_bf16_bits(hf)
    head = EarlyExitHead(_bits_to_gpu(W), max_batch=16)
    K = 128
    tok, prob = head.topk(_bits_to_gpu(h), K)
    assert head.status() == 0
    z64 = orc.head_logits(W, h)
    np.testing.assert_array_equal(head.logits(B).cpu().numpy().astype(np.float64), z64)     # bit-exact logits
    e_tok, e_prob, _ = orc.head_topk(z64, K)
    np.testing.assert_array_equal(tok.cpu().numpy(), e_tok)            # identical selection and order, ties by id
    np.testing.assert_allclose(prob.cpu().numpy(), e_prob, rtol=1e-4, atol=1e-30)      # fp32 underflows below ~1e-38
    np.testing.assert_array_equal(tok[3].cpu().numpy(), np.arange(K))
    head.close()


def test_head_argument_checks():
    from paper_2607_07388_b200 import binding as tfe
    w = torch.zeros((256, 64), dtype=torch.bfloat16, device=DEV)
    for V, d, mb in ((0, 64, 4), (256, 32, 4), (256, 96, 4), (256, 64, 0), (256, 64, 257)):
        with pytest.raises(tfe.TfeError):
            tfe.tfe_head_create(w, V, d, mb)
    hd = tfe.tfe_head_create(w, 256, 64, 8)
    h = torch.zeros((8, 64), dtype=torch.bfloat16, device=DEV)
    t = torch.empty((8, 4), dtype=torch.int32, device=DEV); p = torch.empty((8, 4), dtype=torch.float32, device=DEV)
    for B, K in ((9, 4), (4, 0), (4, 129), (-1, 4)):
        with pytest.raises(tfe.TfeError):
            tfe.tfe_head_topk(hd, h, B, K, t, p)
    tfe.tfe_head_topk(hd, h, 0, 4, t, p)                               # empty batch: nothing to do
    assert tfe.tfe_head_status(hd) == 0
    tfe.tfe_head_destroy(hd)


def test_head_feeds_prefetch_candidates(orc):
    """The chain of Sec. 4.4 on the device: hidden states -> top-K tokens and probabilities (head)
    -> candidate phrases and priorities (tfe_prefetch_candidates), without a host round trip.  The
    head's outputs are checked against the oracle head, and the candidate step against the oracle fed
    with those same tokens and probabilities."""
    import parity_harness as H
    from paper_2607_07388_b200.engine import EarlyExitHead
    w = synth.config(2, n_phrases=60_000, gpu_slots=20_000, B=48)
    tb, pr = H.pair_from_workload(w)
    V, d, B, K = w.vocab, 128, w.B, 32
    rng = np.random.default_rng(17)
    # small-integer weights: fp32 logits are exact, so the head's tokens equal the oracle's
    Wf = rng.integers(-3, 4, size=(V, d)).astype(np.float32)
    hf = rng.integers(-2, 3, size=(B, d)).astype(np.float32)
    # the token that follows each sequence's history in the table stream gets a row aligned with
    # that sequence's hidden state, so it is predicted and its phrases are looked up
    base = tb.safe_len - 3 * B - 16            # late in the stream: rare phrases, mostly outside the GPU tier
    nxt = tb.stream[base + 2 * np.arange(B) + 2]
    for b in range(B):
        Wf[nxt[b]] = 3 * np.sign(hf[b])
    W, h = synth.f32_to_bf16_bits(Wf), synth.f32_to_bf16_bits(hf)
    head = EarlyExitHead(_bits_to_gpu(W), max_batch=B)
    tok, prob = head.topk(_bits_to_gpu(h), K)
    assert head.status() == 0
    e_tok, e_prob, _ = orc.head_topk(orc.head_logits(W, h), K)
    assert (e_tok[:, 0] == nxt).mean() > 0.5
    np.testing.assert_array_equal(tok.cpu().numpy(), e_tok)
    np.testing.assert_allclose(prob.cpu().numpy(), e_prob, rtol=1e-4, atol=1e-30)
    hist = torch.from_numpy(np.stack([tb.stream[base + 2 * b:base + 2 * b + 2] for b in range(B)]).astype(np.int32)).to(DEV)
    ph, tr, sc, sr, cnt = pr.eng.prefetch_candidates(hist, tok, prob, benefit_host=1.0, benefit_ssd=2.0, budget=4096)
    torch.cuda.synchronize()
    # the oracle's chain runs on the oracle head's own outputs (nothing the GPU computed goes into it)
    eph, etr, esc, esr, total = pr.ora.prefetch_candidates(hist.cpu().numpy(), e_tok, e_prob.astype(np.float32),
                                                           benefit_host=1.0, benefit_ssd=2.0, budget=4096)
    n = int(cnt[0].item())
    assert int(cnt[1].item()) == total and n == len(eph) and 5 <= total <= 4096
    # the same candidates (phrase, tier, source); priorities agree to fp32 rounding of the probabilities,
    # so the two orders may differ only among candidates whose priorities are that close
    got = sorted(zip(sr[:n].cpu().numpy().view(np.uint32).tolist(), ph[:n].cpu().numpy().view(np.uint32).tolist(),
                     tr[:n].cpu().numpy().tolist()))
    want = sorted(zip(esr.tolist(), eph.tolist(), etr.tolist()))
    assert got == want
    g_sc = sc[:n].cpu().numpy()
    assert (np.diff(g_sc) <= 0).all()
    by_key = {(s_, p_): v for s_, p_, v in zip(esr.tolist(), eph.tolist(), esc.tolist())}
    for s_, p_, v in zip(sr[:n].cpu().numpy().view(np.uint32).tolist(), ph[:n].cpu().numpy().view(np.uint32).tolist(), g_sc.tolist()):
        assert abs(v - by_key[(s_, p_)]) <= 1e-4 * abs(by_key[(s_, p_)]) + 1e-30
    head.close()
    pr.close()


@pytest.mark.parametrize("seed", range(int(os.environ.get("TFE_RANDOM_CASES", "24"))))
def test_head_random_shapes(orc, seed):
    """Seeded random vocabulary size / width / batch / K, including sizes that leave short last tiles,
    batches that are not multiples of 16 and K up to the limit."""
    from paper_2607_07388_b200.engine import EarlyExitHead
    rng = np.random.default_rng([4404, seed])
    d = int(rng.choice([64, 128, 192, 320, 512, 1024]))
    B = int(rng.choice([1, 2, 15, 16, 17, 48, 64, 100, 128, 200, 256]))
    V = int(rng.integers(8, max(9, min(80_000, 200_000_000 // (d * B)))))
    K = int(rng.integers(1, min(128, V) + 1))
    exact_inputs = bool(rng.random() < 0.4)
    if exact_inputs:                        # small integers: fp32 sums are exact, ties are frequent
        W = synth.f32_to_bf16_bits(rng.integers(-2, 3, size=(V, d)).astype(np.float32))
        h = synth.f32_to_bf16_bits(rng.integers(-2, 3, size=(B, d)).astype(np.float32))
    else:
        W, h = _inputs(seed, V, d, B)
    head = EarlyExitHead(_bits_to_gpu(W), max_batch=B)
    tok, prob = head.topk(_bits_to_gpu(h), K)
    assert head.status() == 0
    z64 = orc.head_logits(W, h)
    if exact_inputs:
        np.testing.assert_array_equal(head.logits(B).cpu().numpy().astype(np.float64), z64)
        e_tok, e_prob, _ = orc.head_topk(z64, K)
        np.testing.assert_array_equal(tok.cpu().numpy(), e_tok)
        np.testing.assert_allclose(prob.cpu().numpy(), e_prob, rtol=1e-4, atol=1e-30)
    else:
        tol = 4e-6 * d * max(np.abs(z64).max(), 1e-6)
        np.testing.assert_allclose(head.logits(B).cpu().numpy(), z64, rtol=0, atol=tol)
        check_topk(z64, tok.cpu().numpy(), prob.cpu().numpy(), K, logit_tol=2 * tol, lse=head.lse(B).cpu().numpy())
    head.close()
