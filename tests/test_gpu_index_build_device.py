"""Index construction on the GPU (tfe_index_build_device): contexts built there must answer every
lookup like the oracle (and so like contexts built on the host), report the same input errors, and
keep the host-side residency mirror that tfe_cache_install relies on."""
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


@pytest.mark.parametrize("orders,load,residency", [((2, 3), 0.7, "all"), ((2, 3, 4), 0.7, "hot_host"),
                                                   ((1, 2, 3, 4), 0.95, "hot_host_ssd"), ((4,), 0.5, "all"),
                                                   ((2, 3), 0.9, "hot_host")])
def test_device_built_index_answers_like_the_oracle(H, orders, load, residency):
    gpu_slots = 30_000 if residency == "all" else 11_000
    w = synth.config(1, B=5, T=301, orders=orders, n_phrases=30_000, gpu_slots=gpu_slots, residency=residency,
                     load_factor=load, p=0.6)
    tb, pr = H.pair_from_workload(w, device_build=True, max_kicks=100_000)
    h = synth.make_hidden_np(w)
    for variant in (0, 1):
        tok = synth.make_queries(w, tb, variant=variant)
        _, ref, info = pr.run_and_compare(tok, h, lam=1.0)
        pr.run_and_compare(tok, h, policy=1, lam=0.5)
    assert info["n_hit"] > 100
    pr.close()


def test_device_and_host_builds_agree_and_install_works(H):
    w = synth.config(1, B=4, T=257, orders=(2, 3, 4), n_phrases=20_000, gpu_slots=8_000, residency="hot_host",
                     reserve_free=300, p=0.7)
    tb, dev_pair = H.pair_from_workload(w, device_build=True)
    _, host_pair = H.pair_from_workload(w)
    tok = synth.make_queries(w, tb)
    h = synth.make_hidden_np(w)
    g_dev, ref, _ = dev_pair.run_and_compare(tok, h, lam=1.0)
    g_host, _, _ = host_pair.run_and_compare(tok, h, lam=1.0)
    for a, b in ((g_dev.sel_phrase, g_host.sel_phrase), (g_dev.sel_slot, g_host.sel_slot), (g_dev.flags, g_host.flags),
                 (g_dev.out.view(torch.int16), g_host.out.view(torch.int16))):
        assert torch.equal(a, b)
    # the host mirror of the residency state is in place: install misses into free slots, then into occupied ones
    want = np.unique(ref.miss_phrase)[:200].astype(np.uint32)
    free = np.nonzero(dev_pair.ora.slot_owner < 0)[0][:100].astype(np.int32)
    used = np.nonzero(dev_pair.ora.slot_owner >= 0)[0][:100].astype(np.int32)
    for ids, dst in ((want[:100], free), (want[100:], used)):
        src = synth.phrase_rows_np(w, ids)
        assert dev_pair.ora.cache_install(ids, src, dst) == 0
        dev_pair.eng.cache_install(ids, src, dst)
        dev_pair.run_and_compare(tok, h, lam=1.0)
    from paper_2607_07388_b200 import binding as tfe
    with pytest.raises(tfe.TfeError):           # already resident: refused from the mirror
        dev_pair.eng.cache_install(want[:1], synth.phrase_rows_np(w, want[:1]), used[:1])
    dev_pair.close(); host_pair.close()


def _try_build(pt, pl, sl, *, vocab=50, orders=(2, 3), C=4, load=0.7, max_kicks=0):
    from paper_2607_07388_b200.engine import Engram
    rows = torch.zeros((C, 16), dtype=torch.bfloat16, device=DEV)
    return Engram(np.asarray(pt, np.int32), np.asarray(pl, np.uint8), np.asarray(sl, np.int32), rows, vocab=vocab,
                  orders=orders, load_factor=load, max_kicks=max_kicks, device_build=True)


def test_device_build_reports_input_errors():
    from paper_2607_07388_b200 import binding as tfe
    pt = [[1, 2, -1, -1], [3, 4, 5, -1], [7, 8, -1, -1]]
    pl, sl = [2, 3, 2], [0, -1, 2]
    _try_build(pt, pl, sl).close()                                     # the good table builds
    cases = [
        (dict(pl=[2, 4, 2]), tfe.TFE_ERR_INVALID_ARG),                 # 4 is not a configured order
        (dict(pl=[2, 0, 2]), tfe.TFE_ERR_INVALID_ARG),
        (dict(pt=[[1, 2, -1, -1], [3, 50, 5, -1], [7, 8, -1, -1]]), tfe.TFE_ERR_INVALID_ARG),   # id = vocab
        (dict(pt=[[1, -1, -1, -1], [3, 4, 5, -1], [7, 8, -1, -1]]), tfe.TFE_ERR_INVALID_ARG),   # padding inside a phrase
        (dict(sl=[0, -3, 2]), tfe.TFE_ERR_INVALID_ARG),
        (dict(sl=[0, 4, 2]), tfe.TFE_ERR_SLOT_RANGE),
        (dict(sl=[2, -1, 2]), tfe.TFE_ERR_SLOT_RANGE),                 # two phrases on one slot
        (dict(pt=[[1, 2, -1, -1], [3, 4, 5, -1], [1, 2, -1, -1]]), tfe.TFE_ERR_DUPLICATE_PHRASE),
    ]
    for change, code in cases:
        args = dict(pt=pt, pl=pl, sl=sl); args.update(change)
        with pytest.raises(tfe.TfeError) as e:
            _try_build(args["pt"], args["pl"], args["sl"])
        assert e.value.status == code, (change, e.value.status)
    # a completely full table cannot be reached with one move per insertion
    many = [[i // 40, i % 40, -1, -1] for i in range(1600)]
    with pytest.raises(tfe.TfeError) as e:
        _try_build(many, [2] * 1600, [-1] * 1600, load=1.0, max_kicks=1)
    assert e.value.status == tfe.TFE_ERR_PROBE_LIMIT
    # an empty table is fine and matches nothing
    eng = _try_build(np.zeros((0, 4)), [], [])
    eng.close()


def test_device_build_full_load_and_duplicates_among_many(H):
    # load 1.0 with room for the moves; one duplicate hidden among 50,000 phrases is found
    w = synth.config(1, orders=(2, 3, 4), n_phrases=50_000, gpu_slots=50_000)
    tb = synth.make_table(w)
    from paper_2607_07388_b200 import binding as tfe
    from paper_2607_07388_b200.engine import Engram
    rows = torch.zeros((w.gpu_slots, 16), dtype=torch.bfloat16, device=DEV)
    eng = Engram(tb.phrase_tokens, tb.phrase_len, tb.init_slot, rows, vocab=w.vocab, orders=w.orders, load_factor=0.97,
                 max_kicks=100_000, device_build=True)
    eng.close()
    pt = tb.phrase_tokens.copy(); pl = tb.phrase_len.copy()
    pt[41_234] = pt[977]; pl[41_234] = pl[977]
    with pytest.raises(tfe.TfeError) as e:
        Engram(pt, pl, tb.init_slot, rows, vocab=w.vocab, orders=w.orders, device_build=True)
    assert e.value.status == tfe.TFE_ERR_DUPLICATE_PHRASE
