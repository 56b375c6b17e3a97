"""Seeded random configurations of the lookup-and-inject call against the oracle: orders, vocabulary
(small ones make every order packed, the large one hashes order 4), row width (including widths that
leave ragged 16-byte steps for a warp), batch shape, query start, policy, gate, lambda, hidden dtype,
in place or not, host- or device-built index, residency mix.  Every case goes through the full
comparison of the harness (integers bit-exact, hidden states within tolerance / bit-exact where the
arithmetic allows)."""
import os

import numpy as np
import pytest
import torch

from paper_2607_07388_b200 import synth

pytestmark = pytest.mark.gpu


def _case(seed):
    rng = np.random.default_rng([2607, seed])
    all_orders = [o for o in (1, 2, 3, 4) if rng.random() < 0.6] or [2]
    vocab = int(rng.choice([37, 500, 4096, synth.VOCAB]))
    d = int(rng.choice([8, 24, 64, 256, 264, 520, 1024, 2048, 4104]))
    shape = "prefill" if rng.random() < 0.6 else "decode"
    n_max = max(all_orders)
    if shape == "prefill":
        B, T = int(rng.integers(1, 7)), int(rng.integers(max(2, n_max), 400))
    else:
        B, T = int(rng.integers(1, 300)), n_max
    # what the tuple space allows (small vocabularies, low orders)
    space = sum(min(vocab ** n, 10 ** 7) for n in all_orders)
    n_phrases = int(min(rng.integers(50, 20_000), max(8, space // 3)))
    residency = str(rng.choice(["all", "hot_host", "hot_host_ssd"]))
    gpu_slots = n_phrases if residency == "all" else max(4, int(n_phrases * rng.uniform(0.2, 0.9)))
    return dict(orders=tuple(all_orders), vocab=vocab, d=d, shape=shape, B=B, T=T, n_phrases=n_phrases,
                residency=residency, gpu_slots=gpu_slots, load=float(rng.choice([0.5, 0.7, 0.9])),
                p=float(rng.uniform(0.2, 0.55 if shape == "prefill" else 0.9)), policy=int(rng.random() < 0.35), gate=int(rng.random() < 0.3),
                lam=float(rng.choice([1.0, 0.5, 2.0, 0.3, 1.7])), hidden=int(rng.random() < 0.25),
                in_place=bool(rng.random() < 0.3), device_build=bool(rng.random() < 0.4), seed=seed)


@pytest.mark.parametrize("seed", range(int(os.environ.get("TFE_RANDOM_CASES", "40"))))
def test_random_configuration(seed):
    import parity_harness as H
    c = _case(seed)
    w = synth.Workload(f"rnd{seed}", 100 + seed, c["shape"], c["B"], c["T"], c["orders"], c["n_phrases"], c["gpu_slots"],
                       d=c["d"], p=c["p"], load_factor=c["load"], residency=c["residency"], rows="gaussian", vocab=c["vocab"])
    try:
        tb = synth.make_table(w)
        tok = synth.make_queries(w, tb)
    except AssertionError as e:                 # e.g. sequences too short to plant that fraction
        pytest.skip(f"inputs not constructible: {e}")
    rows = synth.make_rows_np(w, tb)
    pr = H.Pair(tb.phrase_tokens, tb.phrase_len, tb.init_slot, rows, vocab=w.vocab, orders=w.orders,
                load_factor=w.load_factor, hidden_dtype=c["hidden"], max_kicks=100_000, device_build=c["device_build"])
    if c["hidden"] == 0:
        h = synth.make_hidden_np(w)
    else:
        h = np.random.default_rng(seed).standard_normal((w.Q, w.d)).astype(np.float32)
    q_start = w.q_start
    pr.run_and_compare(tok, h, q_start=q_start, policy=c["policy"], gate=c["gate"], lam=c["lam"], in_place=c["in_place"])
    # and the host-buffer entry point on the same inputs (LONGEST / CONST results must agree with it too)
    if c["policy"] == 0 and c["gate"] == 0 and c["hidden"] == 0:
        from paper_2607_07388_b200 import binding as tfe
        out = np.empty_like(h)
        fl = np.empty(w.Q, np.uint8)
        tfe.tfe_lookup_inject_host(pr.eng.ctx, tok, w.B, w.T, q_start, h, out, lam=c["lam"], flags=fl)
        torch.cuda.synchronize()
        ref = pr.ora.lookup(tok, q_start)
        np.testing.assert_array_equal(fl, ref.flags)
        lam_is_bf16 = (np.float32(c["lam"]).view(np.uint32) & np.uint32(0xFFFF)) == 0
        if lam_is_bf16:
            _, rounded = pr.ora.inject(ref, h, lam=c["lam"])
            np.testing.assert_array_equal(out, rounded)
    pr.close()
