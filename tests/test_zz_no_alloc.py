"""The allocation-free lookup entry point against the ordinary one.

Some embedders of this library cannot let it call cudaMalloc: an inference server that has
already given every free byte of device memory to its own pool (an allocation would fail), or a
decode loop that cannot take the device-wide stall an allocation or a free causes.  For them
``tfe_lookup_inject_noalloc`` runs the same kernels on a fixed scratch area inside the library
image and writes the miss list into buffers the caller owns.  This test calls it through the C ABI
twice in a row and requires the same results as ``tfe_lookup_inject`` + ``tfe_miss_list``; a second
test checks it against the CPU oracle over a sequence of calls that share the fixed area (a large call
with every order reported, a small one from another context, an empty one, a refused one).  The
file sorts last so that a run stopping at the first failure has already run everything else.
"""
import numpy as np
import pytest
import torch

from paper_2607_07388_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _setup(policy_orders=(2, 3, 4)):
    from paper_2607_07388_b200 import build
    build.build()
    from paper_2607_07388_b200 import binding as tfe
    from paper_2607_07388_b200.engine import Engram, bf16_tensor_from_bits
    w = synth.config(3, n_phrases=40_000, gpu_slots=30_000, residency="hot_host_ssd", B=3, T=1500, d=1024,
                     orders=policy_orders, p=0.4, rows="procedural")
    tb = synth.make_table(w)
    rows = bf16_tensor_from_bits(synth.make_rows_np(w, tb), DEV)
    eng = Engram(tb.phrase_tokens, tb.phrase_len, tb.init_slot, rows, vocab=w.vocab, orders=w.orders)
    tok = torch.from_numpy(synth.make_queries(w, tb)).to(DEV)
    h = synth.make_hidden_torch(w, DEV)
    return tfe, w, eng, rows, tok, h


@pytest.mark.parametrize("policy,gate,lam", [(0, 0, 1.0), (0, 0, 0.3), (1, 1, 0.7)])
def test_noalloc_entry_matches_the_ordinary_lookup_twice_in_a_row(policy, gate, lam):
    tfe, w, eng, rows, tok, h = _setup()
    cols = len(w.orders) if policy == 1 else 1
    ent = w.Q * cols
    # reference: the ordinary entry point (context-owned scratch and miss list)
    ref = eng.lookup_inject(tok, h, policy=policy, gate=gate, lam=lam)
    rq, rp, rt, rcnt = eng.miss_list()
    assert rcnt > 20 and int((ref.flags == 1).sum()) > 200
    shape = (w.Q,) if policy == 0 else (w.Q, cols)
    for round_no in range(2):
        out = torch.full_like(h, float("nan"))
        sp = torch.full(shape, -7, dtype=torch.int32, device=DEV)
        ss = torch.full(shape, -7, dtype=torch.int32, device=DEV)
        fl = torch.full(shape, 9, dtype=torch.uint8, device=DEV)
        mq = torch.full((ent,), -1, dtype=torch.int32, device=DEV)
        mp = torch.full((ent,), -1, dtype=torch.int32, device=DEV)
        mt = torch.full((ent,), 9, dtype=torch.uint8, device=DEV)
        mc = torch.full((1,), 12345, dtype=torch.int32, device=DEV)
        tfe.tfe_lookup_inject_noalloc(eng.ctx, tok, w.B, w.T, 0, h, out, policy=policy, gate=gate, lam=lam,
                                      sel_phrase=sp, sel_slot=ss, flags=fl, miss_q=mq, miss_phrase=mp,
                                      miss_tier=mt, miss_count=mc)
        torch.cuda.synchronize()
        assert torch.equal(sp, ref.sel_phrase) and torch.equal(ss, ref.sel_slot) and torch.equal(fl, ref.flags)
        n = int(mc.item())
        assert n == rcnt
        np.testing.assert_array_equal(mq[:n].cpu().numpy().view(np.uint32), rq)
        np.testing.assert_array_equal(mp[:n].cpu().numpy().view(np.uint32), rp)
        np.testing.assert_array_equal(mt[:n].cpu().numpy(), rt)
        # same kernels, same inputs: the hidden states agree to the tolerance of the parity tests (2e-2)
        # and in fact bit for bit
        err = (out.float() - ref.out.float()).abs().max().item()
        assert err <= 2e-2, err
        assert torch.equal(out.view(torch.int16), ref.out.view(torch.int16)), round_no
    eng.close()


def test_noalloc_entry_refuses_calls_beyond_its_fixed_scratch():
    tfe, w, eng, rows, tok, h = _setup()
    Bbig = tfe.NOALLOC_MAX_ENTRIES // 4 + 1          # one query too many at T = 4, q_start = 0
    big_tok = torch.zeros((Bbig, 4), dtype=torch.int32, device=DEV)
    dummy = torch.zeros(16, dtype=torch.int32, device=DEV)
    with pytest.raises(tfe.TfeError) as ei:
        tfe.tfe_lookup_inject_noalloc(eng.ctx, big_tok, Bbig, 4, 0, dummy, dummy, miss_q=dummy, miss_phrase=dummy,
                                      miss_tier=dummy, miss_count=dummy)
    assert ei.value.status == tfe.TFE_ERR_CAPACITY
    with pytest.raises(tfe.TfeError) as ei:          # the miss buffers are not optional
        tfe.tfe_lookup_inject_noalloc(eng.ctx, tok, w.B, w.T, 0, h, torch.empty_like(h), miss_q=None,
                                      miss_phrase=dummy, miss_tier=dummy, miss_count=dummy)
    assert ei.value.status == tfe.TFE_ERR_INVALID_ARG
    eng.close()


def _noalloc_against_oracle(tfe, pr, tok_np, h_bits, *, policy, gate, lam, q_start=0):
    """One call of the allocation-free entry point on the table of `pr`, every output against the oracle."""
    import parity_harness as H
    from paper_2607_07388_b200.engine import bf16_tensor_from_bits, bits_from_bf16_tensor
    B, T = tok_np.shape
    Q = B * (T - q_start)
    cols = len(pr.orders) if policy == 1 else 1
    shape = (Q,) if policy == 0 else (Q, cols)
    tok = torch.from_numpy(np.ascontiguousarray(tok_np, np.int32)).to(DEV)
    h = bf16_tensor_from_bits(h_bits, DEV) if Q else torch.zeros((0, pr.d), dtype=torch.bfloat16, device=DEV)
    out = torch.full_like(h, float("nan"))
    sp = torch.full(shape, -7, dtype=torch.int32, device=DEV)
    ss = torch.full(shape, -7, dtype=torch.int32, device=DEV)
    fl = torch.full(shape, 9, dtype=torch.uint8, device=DEV)
    ent = max(1, Q * cols)
    mq = torch.full((ent,), -1, dtype=torch.int32, device=DEV)
    mp = torch.full((ent,), -1, dtype=torch.int32, device=DEV)
    mt = torch.full((ent,), 9, dtype=torch.uint8, device=DEV)
    mc = torch.full((1,), 12345, dtype=torch.int32, device=DEV)
    tfe.tfe_lookup_inject_noalloc(pr.eng.ctx, tok, B, T, q_start, h, out, policy=policy, gate=gate, lam=lam,
                                  sel_phrase=sp, sel_slot=ss, flags=fl, miss_q=mq, miss_phrase=mp,
                                  miss_tier=mt, miss_count=mc)
    torch.cuda.synchronize()
    n = int(mc.item())
    if Q == 0:
        assert n == 0
        return 0, 0
    ref = pr.ora.lookup(np.ascontiguousarray(tok_np, np.int32), q_start, policy, "sorted")
    exact, rounded = pr.ora.inject(ref, h_bits, policy=policy, gate=gate, lam=float(np.float32(lam)))
    np.testing.assert_array_equal(sp.cpu().numpy().view(np.uint32), ref.sel_phrase)
    np.testing.assert_array_equal(ss.cpu().numpy(), ref.sel_slot)
    np.testing.assert_array_equal(fl.cpu().numpy(), ref.flags)
    assert n == len(ref.miss_q)
    np.testing.assert_array_equal(mq[:n].cpu().numpy().view(np.uint32), ref.miss_q)
    np.testing.assert_array_equal(mp[:n].cpu().numpy().view(np.uint32), ref.miss_phrase)
    np.testing.assert_array_equal(mt[:n].cpu().numpy(), ref.miss_tier)
    got = bits_from_bf16_tensor(out)
    touched = (ref.flags.reshape(Q, -1) == 1).any(axis=1)
    np.testing.assert_array_equal(got[~touched], h_bits[~touched])
    err = np.abs(synth.bf16_bits_to_f32(got).astype(np.float64) - exact).max()
    assert err <= H.TOL_BF16, err
    if policy == 0 and gate == 0 and (np.float32(lam).view(np.uint32) & np.uint32(0xFFFF)) == 0:
        np.testing.assert_array_equal(got, rounded)      # one rounding of the exact value on both sides
    return int(touched.sum()), n


def test_noalloc_entry_against_the_oracle_over_calls_that_share_the_area():
    """The fixed area keeps what the last call left, whichever context made it.  A large call that reports
    every order (three records per query), then a small longest-match call from a SECOND context over
    another table, then an empty call, then a refused call, then the first context again: every one of
    them must give the oracle's results, so nothing a call leaves behind may leak into the next."""
    from paper_2607_07388_b200 import build
    build.build()
    from oracle import tfe_oracle
    tfe_oracle.build()
    import parity_harness as H
    from paper_2607_07388_b200 import binding as tfe
    w1 = synth.config(3, n_phrases=40_000, gpu_slots=30_000, residency="hot_host_ssd", B=3, T=1500, d=1024,
                      orders=(2, 3, 4), p=0.4, rows="procedural")
    w2 = synth.config(2, n_phrases=20_000, gpu_slots=6_000, B=48, d=256, rows="procedural")
    tb1, pr1 = H.pair_from_workload(w1)
    tb2, pr2 = H.pair_from_workload(w2)
    tok1, h1 = synth.make_queries(w1, tb1), synth.make_hidden_np(w1)
    tok2, h2 = synth.make_queries(w2, tb2), synth.make_hidden_np(w2)
    hits, misses = _noalloc_against_oracle(tfe, pr1, tok1, h1, policy=1, gate=0, lam=0.5)
    assert hits > 200 and misses > 20
    hits, misses = _noalloc_against_oracle(tfe, pr2, tok2, h2, policy=0, gate=0, lam=1.0, q_start=w2.q_start)
    assert hits > 0 and misses > 0
    _noalloc_against_oracle(tfe, pr2, tok2[:0], h2[:0], policy=0, gate=0, lam=1.0, q_start=w2.q_start)
    dummy = torch.zeros(16, dtype=torch.int32, device=DEV)
    with pytest.raises(tfe.TfeError):                    # refused before anything of the shared area is touched
        tfe.tfe_lookup_inject_noalloc(pr2.eng.ctx, torch.from_numpy(tok2).to(DEV), w2.B, w2.T, w2.q_start, None, None,
                                      miss_q=dummy, miss_phrase=dummy, miss_tier=dummy, miss_count=dummy)
    hits, misses = _noalloc_against_oracle(tfe, pr1, tok1, h1, policy=0, gate=0, lam=1.0)
    assert hits > 200 and misses > 20
    _noalloc_against_oracle(tfe, pr1, tok1, h1, policy=0, gate=1, lam=0.7)
    pr1.close()
    pr2.close()
