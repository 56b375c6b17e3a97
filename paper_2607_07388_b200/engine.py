"""A small convenience layer over the C-ABI binding: owns a context and the
result tensors, so a caller writes ``eng.lookup_inject(tokens, h)``.

Nothing is computed here -- every call goes straight to libtfe.so.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np
import torch

from . import binding as tfe


@dataclass
class LookupOutput:
    out: torch.Tensor          # [Q, d] hidden dtype
    sel_phrase: torch.Tensor   # uint32 bit patterns in an int32 tensor, [Q] or [Q, n_orders]
    sel_slot: torch.Tensor     # int32
    flags: torch.Tensor        # uint8


class Engram:
    """GPU-resident phrase index + GPU-tier row store for one table."""

    def __init__(self, phrase_tokens, phrase_len, init_slot, gpu_rows: torch.Tensor, *, vocab, orders,
                 load_factor=0.7, hidden_dtype=tfe.HIDDEN_BF16, max_kicks=0, stream=None, device_build=False):
        assert gpu_rows.is_cuda and gpu_rows.dtype == torch.bfloat16 and gpu_rows.is_contiguous()
        self.rows = gpu_rows
        self.C, self.d = gpu_rows.shape
        self.orders = tuple(int(o) for o in orders)
        self.hidden_dtype = hidden_dtype
        self.torch_hidden = torch.bfloat16 if hidden_dtype == tfe.HIDDEN_BF16 else torch.float32
        self.cfg = tfe.make_config(d=self.d, vocab=vocab, orders=self.orders, n_phrases=len(phrase_len),
                                   gpu_slots=self.C, load_factor=load_factor, hidden_dtype=hidden_dtype,
                                   max_kicks=max_kicks)
        self.ctx = 0
        if device_build:        # the phrase arrays go to (or already are on) the device; the index is built there
            dev = gpu_rows.device
            as_dev = lambda a, dt: a.to(dev, dt).contiguous() if torch.is_tensor(a) else \
                torch.from_numpy(np.ascontiguousarray(a)).to(dev, dt)
            pt = as_dev(phrase_tokens, torch.int32).reshape(-1, 4)
            pl = as_dev(phrase_len, torch.uint8)
            sl = as_dev(init_slot, torch.int32)
            self.ctx = tfe.tfe_index_build_device(self.cfg, pt, pl, sl, gpu_rows, stream)
        else:
            self.ctx = tfe.tfe_index_build(self.cfg, phrase_tokens, phrase_len, init_slot, gpu_rows, stream)

    def close(self):
        if getattr(self, "ctx", 0):
            tfe.tfe_destroy(self.ctx)
            self.ctx = 0

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def lookup_inject(self, tokens: torch.Tensor, h: torch.Tensor, out: torch.Tensor | None = None, *,
                      q_start=0, policy=tfe.POLICY_LONGEST, gate=tfe.GATE_CONST, lam=1.0, want_sel=True,
                      stream=None) -> LookupOutput:
        B, T = tokens.shape
        Q = B * (T - q_start)
        assert tokens.dtype == torch.int32 and tokens.is_cuda
        assert h.shape == (Q, self.d) and h.dtype == self.torch_hidden
        if out is None:
            out = torch.empty_like(h)
        shape = (Q,) if policy == tfe.POLICY_LONGEST else (Q, len(self.orders))
        sp = ss = fl = None
        if want_sel:
            sp = torch.empty(shape, dtype=torch.int32, device=h.device)
            ss = torch.empty(shape, dtype=torch.int32, device=h.device)
            fl = torch.empty(shape, dtype=torch.uint8, device=h.device)
        tfe.tfe_lookup_inject(self.ctx, tokens, B, T, q_start, h, out, policy=policy, gate=gate, lam=lam,
                              sel_phrase=sp, sel_slot=ss, flags=fl, stream=stream)
        return LookupOutput(out, sp, ss, fl)

    def miss_list(self, cap: int | None = None, stream=None, allow_overflow=False):
        if cap is None:
            cap = 1 << 20
        return tfe.tfe_miss_list(self.ctx, cap, stream, allow_overflow)

    def prefetch_candidates(self, history: torch.Tensor, cand_tokens: torch.Tensor, cand_prob: torch.Tensor, *,
                            usefulness: torch.Tensor | None = None, benefit_host=1.0, benefit_ssd=2.0, budget=4096,
                            stream=None):
        """(phrase, tier, score, src, [written, found]) device tensors of the `budget` best candidates."""
        B, H = history.shape
        K = cand_tokens.shape[1]
        dev = cand_tokens.device
        ph = torch.empty(max(budget, 1), dtype=torch.int32, device=dev)
        tr = torch.empty(max(budget, 1), dtype=torch.uint8, device=dev)
        sc = torch.empty(max(budget, 1), dtype=torch.float32, device=dev)
        sr = torch.empty(max(budget, 1), dtype=torch.int32, device=dev)
        cnt = torch.zeros(2, dtype=torch.int32, device=dev)
        tfe.tfe_prefetch_candidates(self.ctx, history, B, H, cand_tokens, cand_prob, K, out_phrase=ph, out_tier=tr,
                                    out_score=sc, out_src=sr, out_count=cnt, usefulness=usefulness,
                                    benefit_host=benefit_host, benefit_ssd=benefit_ssd, budget=budget, stream=stream)
        return ph, tr, sc, sr, cnt

    def cache_install(self, phrase_ids, src_rows, dst_slots, stream=None):
        tfe.tfe_cache_install(self.ctx, phrase_ids, src_rows, dst_slots, stream)

    def cache_install_device(self, phrase_ids: torch.Tensor, src_rows: torch.Tensor, dst_slots: torch.Tensor, stream=None):
        """Device tensors in, (applied uint8 [n], count int32 [1]) device tensors out; nothing synchronises."""
        n = int(phrase_ids.shape[0])
        applied = torch.empty(max(n, 1), dtype=torch.uint8, device=phrase_ids.device)
        count = torch.zeros(1, dtype=torch.int32, device=phrase_ids.device)
        tfe.tfe_cache_install_device(self.ctx, n, phrase_ids, src_rows, dst_slots, applied, count, stream)
        return applied[:n], count

    def cache_policy_enable(self, stream=None):
        tfe.tfe_cache_policy_enable(self.ctx, stream)

    def cache_select_victims(self, n, half_life=0, stream=None):
        return tfe.tfe_cache_select_victims(self.ctx, n, half_life, stream)

    def cache_stats(self, stream=None):
        return tfe.tfe_cache_stats(self.ctx, self.C, stream)


def bf16_tensor_from_bits(bits: np.ndarray, device) -> torch.Tensor:
    """uint16 bit patterns -> torch.bfloat16 tensor on ``device`` (no conversion)."""
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).to(device).view(torch.bfloat16)


def bits_from_bf16_tensor(t: torch.Tensor) -> np.ndarray:
    return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


class EarlyExitHead:
    """softmax(W_pref h) + top-K on the GPU.  ``w_pref``: bf16 CUDA tensor [V, d], kept alive here."""

    def __init__(self, w_pref: torch.Tensor, max_batch: int = 256):
        assert w_pref.is_cuda and w_pref.dtype == torch.bfloat16 and w_pref.is_contiguous()
        self.w = w_pref
        self.V, self.d = w_pref.shape
        self.max_batch = max_batch
        self.handle = tfe.tfe_head_create(w_pref, self.V, self.d, max_batch)

    def close(self):
        if getattr(self, "handle", 0):
            tfe.tfe_head_destroy(self.handle)
            self.handle = 0

    def __del__(self):
        try:
            self.close()
        except Exception:       # interpreter shutdown: the binding may be gone already
            pass

    def topk(self, hidden: torch.Tensor, K: int, stream=None):
        """(tokens int32 [B, K], prob float32 [B, K]) on the device."""
        assert hidden.is_cuda and hidden.dtype == torch.bfloat16 and hidden.is_contiguous()
        B = hidden.shape[0]
        tokens = torch.empty((B, K), dtype=torch.int32, device=hidden.device)
        prob = torch.empty((B, K), dtype=torch.float32, device=hidden.device)
        tfe.tfe_head_topk(self.handle, hidden, B, K, tokens, prob, stream)
        return tokens, prob

    def logits(self, B: int) -> torch.Tensor:
        """fp32 [B, V] copy of the logits of the most recent call (synchronises)."""
        addr, ld, _ = tfe.tfe_head_buffers(self.handle)
        torch.cuda.synchronize()
        return _device_view(addr, (B, ld), "<f4", self.w.device)[:, :self.V].clone()

    def lse(self, B: int) -> torch.Tensor:
        _, _, addr = tfe.tfe_head_buffers(self.handle)
        torch.cuda.synchronize()
        return _device_view(addr, (B,), "<f4", self.w.device).clone()

    def status(self) -> int:
        return tfe.tfe_head_status(self.handle)


class _DevicePointer:
    def __init__(self, ptr, shape, typestr):
        self.__cuda_array_interface__ = {"shape": tuple(shape), "typestr": typestr, "data": (ptr, False), "version": 2}


def _device_view(ptr: int, shape, typestr: str, device) -> torch.Tensor:
    """A tensor over library-owned device memory (no copy, no ownership)."""
    return torch.as_tensor(_DevicePointer(ptr, shape, typestr), device=device)


class MinedPhrases:
    """Result of mine_ngrams: device tensors cut to the entries written, plus the host-side totals."""

    def __init__(self, tokens, length, count, n_found, distinct, hist):
        self.phrase_tokens, self.phrase_len, self.count = tokens, length, count
        self.n_found, self.distinct, self.hist = n_found, distinct, hist

    def __len__(self):
        return self.phrase_len.numel()


def mine_ngrams(corpus: torch.Tensor, *, vocab: int, orders, min_count: int = 2, cap: int, want_hist: bool = True,
                workspace: torch.Tensor | None = None, stream=None) -> MinedPhrases:
    """Every n-gram of `corpus` (device int32 [L]) that occurs at least `min_count` times, in order of first
    occurrence; `count` holds uint32 values in an int32 tensor.  The result feeds Engram(device_build=True).
    `workspace`: a device uint8 tensor of tfe_mine_workspace_bytes(L, n_orders) bytes kept by the caller across
    calls (None: the library allocates and frees its own)."""
    assert corpus.is_cuda and corpus.dtype == torch.int32 and corpus.is_contiguous()
    dev = corpus.device
    pt = torch.empty((max(cap, 1), 4), dtype=torch.int32, device=dev)
    pl = torch.empty(max(cap, 1), dtype=torch.uint8, device=dev)
    pc = torch.empty(max(cap, 1), dtype=torch.int32, device=dev)
    n_found, distinct, hist = tfe.tfe_mine_ngrams(corpus, corpus.numel(), vocab, orders, min_count, cap, pt, pl, pc,
                                                  want_hist=want_hist, workspace=workspace,
                                                  workspace_bytes=0 if workspace is None else workspace.numel(),
                                                  stream=stream)
    n = min(n_found, cap)
    return MinedPhrases(pt[:n], pl[:n], pc[:n], n_found, distinct, hist)


def assign_residency(count: torch.Tensor, gpu_slots: int, host_min_count: int = 2, stream=None):
    """(init_slot int32 [N] on the device, (n_gpu, n_host, n_ssd)): the gpu_slots most frequent phrases start in
    the GPU tier (equal counts: smaller id first; slots in id order), the rest is tagged host or SSD by count."""
    assert count.is_cuda and count.dtype == torch.int32 and count.is_contiguous()
    init_slot = torch.empty(max(count.numel(), 1), dtype=torch.int32, device=count.device)
    tiers = tfe.tfe_assign_residency(count, count.numel(), gpu_slots, host_min_count, init_slot, stream)
    return init_slot[:count.numel()], tiers
