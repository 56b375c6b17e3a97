"""The allocation-free lookup entry point against the ordinary one.

Some embedders of this library cannot let it call cudaMalloc: an inference server that has
already given every free byte of device memory to its own pool (an allocation would fail), or a
decode loop that cannot take the device-wide stall an allocation or a free causes.  For them
``tfe_lookup_inject_noalloc`` runs the same kernels on a fixed scratch area inside the library
image and writes the miss list into buffers the caller owns.  This test calls it through the C ABI
twice in a row and requires the same results as ``tfe_lookup_inject`` + ``tfe_miss_list``.  The
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
