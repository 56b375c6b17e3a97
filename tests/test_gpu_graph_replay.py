"""A captured lookup replayed on new contents.

The library keeps its launch state on the device (counters, the call's record tag, the miss list), so a
`tfe_lookup_inject` captured in a CUDA graph can be replayed unchanged: this is how a serving loop issues a
fixed-shape step, and how the benchmark times its headline region.  Here a graph holding one call -- and one
holding three calls back to back on different buffers -- is replayed after the token and hidden-state buffers
have been overwritten, and every replay is checked against the oracle: selections, flags, the miss list read
after the replay, and the hidden states."""
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


def _expect(H, pr, tok, h, q_start, lam):
    ref = pr.ora.lookup(np.ascontiguousarray(tok, np.int32), q_start, 0, "sorted")
    exact, rounded = pr.ora.inject(ref, h, lam=float(np.float32(lam)))
    return ref, exact, rounded


def _compare(H, got_sel, got_out, ref, rounded):
    sp, ss, fl = got_sel
    np.testing.assert_array_equal(sp.cpu().numpy().view(np.uint32), ref.sel_phrase)
    np.testing.assert_array_equal(ss.cpu().numpy(), ref.sel_slot)
    np.testing.assert_array_equal(fl.cpu().numpy(), ref.flags)
    np.testing.assert_array_equal(H.bits_from_bf16_tensor(got_out), rounded)     # lambda = 1: one rounding on both sides


@pytest.mark.parametrize("shape", ["prefill", "decode"])
def test_captured_lookup_replays_on_fresh_contents(H, shape):
    from paper_2607_07388_b200 import binding as tfe
    from paper_2607_07388_b200.engine import bf16_tensor_from_bits
    if shape == "prefill":
        w = synth.config(3, n_phrases=40_000, gpu_slots=30_000, residency="hot_host_ssd", B=3, T=1500, d=1024,
                         orders=(2, 3, 4), p=0.4, rows="procedural")
    else:
        w = synth.config(2, n_phrases=40_000, gpu_slots=12_000, B=64, d=1024, rows="procedural")
    tb, pr = H.pair_from_workload(w)
    ctx, q0, Q = pr.eng.ctx, w.q_start, w.Q
    n_sets = 3
    toks = [torch.zeros((w.B, w.T), dtype=torch.int32, device=H.DEV) for _ in range(n_sets)]
    hs = [torch.zeros((Q, w.d), dtype=torch.bfloat16, device=H.DEV) for _ in range(n_sets)]
    outs = [torch.zeros_like(hs[0]) for _ in range(n_sets)]
    sels = [(torch.zeros(Q, dtype=torch.int32, device=H.DEV), torch.zeros(Q, dtype=torch.int32, device=H.DEV),
             torch.zeros(Q, dtype=torch.uint8, device=H.DEV)) for _ in range(n_sets)]

    def call(k, stream):
        tfe.tfe_lookup_inject(ctx, toks[k], w.B, w.T, q0, hs[k], outs[k], lam=1.0, sel_phrase=sels[k][0],
                              sel_slot=sels[k][1], flags=sels[k][2], stream=stream)

    call(0, None)                                   # sizes the context's buffers outside the capture
    torch.cuda.synchronize()
    cs = torch.cuda.Stream()
    one, three = torch.cuda.CUDAGraph(), torch.cuda.CUDAGraph()
    with torch.cuda.graph(one, stream=cs):
        call(0, cs)
    with torch.cuda.graph(three, stream=cs):
        for k in range(n_sets):
            call(k, cs)
    total_hits = total_misses = 0
    for rep in range(3):
        fresh = []
        for k in range(n_sets):
            v = 10 * rep + k + 1
            tok_np, h_np = synth.make_queries(w, tb, variant=v), synth.make_hidden_np(w, variant=v)
            toks[k].copy_(torch.from_numpy(tok_np))
            hs[k].copy_(bf16_tensor_from_bits(h_np, H.DEV))
            outs[k].fill_(float("nan"))
            fresh.append((tok_np, h_np))
        torch.cuda.synchronize()
        # one captured call
        one.replay()
        mq, mp, mt, cnt = pr.eng.miss_list()
        ref, _, rounded = _expect(H, pr, *fresh[0], q0, 1.0)
        _compare(H, sels[0], outs[0], ref, rounded)
        assert cnt == len(ref.miss_q)
        np.testing.assert_array_equal(mq, ref.miss_q)
        np.testing.assert_array_equal(mp, ref.miss_phrase)
        np.testing.assert_array_equal(mt, ref.miss_tier)
        total_hits += int((ref.flags == 1).sum())
        total_misses += int(cnt)
        # three captured calls back to back: outputs of every one, miss list of the last
        for k in range(n_sets):
            outs[k].fill_(float("nan"))
        three.replay()
        mq, mp, mt, cnt = pr.eng.miss_list()
        for k in range(n_sets):
            ref, _, rounded = _expect(H, pr, *fresh[k], q0, 1.0)
            _compare(H, sels[k], outs[k], ref, rounded)
        assert cnt == len(ref.miss_q)
        np.testing.assert_array_equal(mq, ref.miss_q)
        np.testing.assert_array_equal(mp, ref.miss_phrase)
        np.testing.assert_array_equal(mt, ref.miss_tier)
    assert total_hits > 30 and total_misses > 10
    pr.close()
