"""Shared helpers for the GPU parity tests: drive libcart.so through the binding from a synthetic
workload and mirror the same state into the CPU oracle's bookkeeping."""
from __future__ import annotations

from typing import List, Optional, Sequence

import numpy as np
import torch

import oracle
from paper_2506_06266_b200 import binding, buildlib, synth

# Tolerances the benchmark contract states for bf16 outputs with fp32 accumulation.
TOL_MAX_ABS = 2e-2
TOL_REL_FRO = 1e-2
TOL_LSE = 1e-3


def ensure_built():
    buildlib.build()
    return binding.load_library()


def to_f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().to(torch.float64).cpu().numpy()


def assert_close(out_gpu: torch.Tensor, lse_gpu: Optional[torch.Tensor], out_ref: np.ndarray,
                 lse_ref: np.ndarray, what: str = "") -> dict:
    o = to_f64(out_gpu)
    assert np.all(np.isfinite(o)), what + ": non-finite output"
    diff = o - out_ref
    max_abs = float(np.max(np.abs(diff)))
    rel = float(np.linalg.norm(diff) / max(np.linalg.norm(out_ref), 1e-300))
    res = {"max_abs": max_abs, "rel_fro": rel}
    assert max_abs <= TOL_MAX_ABS, "%s: max abs error %.3e" % (what, max_abs)
    assert rel <= TOL_REL_FRO, "%s: relative (Frobenius) error %.3e" % (what, rel)
    if lse_gpu is not None:
        dl = float(np.max(np.abs(to_f64(lse_gpu) - lse_ref)))
        res["lse"] = dl
        assert dl <= TOL_LSE, "%s: lse error %.3e" % (what, dl)
    return res


class Session:
    """An arena, a context and the handles of one workload on the GPU; optionally the same state in
    an ``oracle.OracleCache``."""

    def __init__(self, n_layers: int, n_q_heads: int, n_kv_heads: int, arena_bytes: int,
                 max_requests: int = 64, max_cartridges: int = 64, device: str = "cuda:0",
                 with_oracle: bool = True, scale: float = 0.0, max_parts: int = 0,
                 arena_fill: Optional[int] = None):
        ensure_built()
        self.dev = torch.device(device)
        self.L, self.Hq, self.Hkv = n_layers, n_q_heads, n_kv_heads
        self.cfg = binding.make_config(n_layers, n_q_heads, n_kv_heads, max_requests, max_cartridges,
                                       device=self.dev.index or 0, softmax_scale=scale, max_parts=max_parts)
        self.scratch = binding.cart_scratch_bytes(self.cfg)
        total = self.scratch + int(arena_bytes) + 256
        self.arena = torch.empty(total, dtype=torch.uint8, device=self.dev)
        if arena_fill is not None:
            self.arena.view(torch.int16).fill_(arena_fill)
            torch.cuda.synchronize(self.dev)
        self.cfg.arena = self.arena.data_ptr()
        self.cfg.arena_bytes = total
        self.ctx = binding.cart_create(self.cfg)
        eff_scale = scale if scale > 0 else 128 ** -0.5
        self.oc = oracle.OracleCache(n_layers, n_q_heads, n_kv_heads, 128, eff_scale) if with_oracle else None
        self.cart_map = {}   # gpu cartridge id -> oracle id
        self.req_map = {}    # gpu request id -> oracle id

    # -- state ------------------------------------------------------------------------------
    def register(self, k: torch.Tensor, v: torch.Tensor) -> int:
        k, v = k.to(self.dev).contiguous(), v.to(self.dev).contiguous()
        cid = binding.cart_register_cartridge(self.ctx, k, v, k.shape[2])
        torch.cuda.synchronize(self.dev)
        if self.oc is not None:
            self.cart_map[cid] = self.oc.register(synth.bits(k), synth.bits(v))
        return cid

    def compose(self, parts: Sequence[int]) -> int:
        cid = binding.cart_compose(self.ctx, parts)
        if self.oc is not None:
            self.cart_map[cid] = self.oc.compose([self.cart_map[p] for p in parts])
        return cid

    def open(self, cart: int, capacity: int, paged: bool = False) -> int:
        rid = (binding.cart_request_open_paged if paged else binding.cart_request_open)(self.ctx, cart, capacity)
        if self.oc is not None:
            self.req_map[rid] = self.oc.open(None if cart == binding.CART_NONE else self.cart_map[cart])
        return rid

    def extend(self, req: int, k: torch.Tensor, v: torch.Tensor) -> None:
        """k, v: bf16 [L][T][Hkv][128]; appended to every layer."""
        k, v = k.to(self.dev).contiguous(), v.to(self.dev).contiguous()
        T = k.shape[1]
        if T == 0:
            return
        for layer in range(self.L):
            binding.cart_extend_kv(self.ctx, layer, req, k[layer], v[layer], T)
        torch.cuda.synchronize(self.dev)
        if self.oc is not None:
            kb, vb = synth.bits(k), synth.bits(v)
            for layer in range(self.L):
                self.oc.extend(layer, self.req_map[req], kb[layer], vb[layer])

    def append(self, layer: int, reqs: Sequence[int], k_new: torch.Tensor, v_new: torch.Tensor) -> None:
        """k_new, v_new: bf16 [len(reqs)][Hkv][128]."""
        k_new, v_new = k_new.to(self.dev).contiguous(), v_new.to(self.dev).contiguous()
        binding.cart_append_kv(self.ctx, layer, reqs, k_new, v_new)
        if self.oc is not None:
            torch.cuda.synchronize(self.dev)
            self.oc.append(layer, [self.req_map[r] for r in reqs], synth.bits(k_new), synth.bits(v_new))

    def decode(self, layer: int, reqs: Sequence[int], q: torch.Tensor, want_lse: bool = True):
        q = q.to(self.dev).contiguous()
        out = torch.full_like(q, float("nan"))
        lse = torch.full(q.shape[:2], float("nan"), dtype=torch.float32, device=self.dev) if want_lse else None
        binding.cart_decode_attention(self.ctx, layer, reqs, q, out, lse)
        binding.cart_sync_status(self.ctx)
        return out, lse

    def decode_step(self, layer: int, reqs: Sequence[int], k_new: torch.Tensor, v_new: torch.Tensor,
                    q: torch.Tensor):
        """Fused append + decode on the GPU; the oracle's bookkeeping gets the same append."""
        k_new, v_new, q = k_new.to(self.dev).contiguous(), v_new.to(self.dev).contiguous(), q.to(self.dev).contiguous()
        out = torch.full_like(q, float("nan"))
        lse = torch.full(q.shape[:2], float("nan"), dtype=torch.float32, device=self.dev)
        binding.cart_decode_step(self.ctx, layer, reqs, k_new, v_new, q, out, lse)
        binding.cart_sync_status(self.ctx)
        if self.oc is not None:
            self.oc.append(layer, [self.req_map[r] for r in reqs], synth.bits(k_new), synth.bits(v_new))
        return out, lse

    def oracle_decode(self, layer: int, reqs: Sequence[int], q: torch.Tensor):
        return self.oc.decode(layer, [self.req_map[r] for r in reqs], synth.bits(q))

    def decode_and_check(self, layer: int, reqs: Sequence[int], q: torch.Tensor, what: str = "") -> dict:
        out, lse = self.decode(layer, reqs, q)
        ro, rl = self.oracle_decode(layer, reqs, q)
        return assert_close(out, lse, ro, rl, what or "layer %d" % layer)

    def close(self):
        if self.ctx:
            binding.cart_destroy(self.ctx)
            self.ctx = 0
        self.arena = None


def workload_arena_bytes(w: synth.Workload, extra_capacity: int = 0) -> int:
    per_tok = w.n_layers * w.kv_bytes_per_token_layer()
    caps = [-(-(int(s) + extra_capacity) // 64) * 64 for s in w.suffix_lengths()]
    return w.n_cartridges * w.p * per_tok + sum(caps) * per_tok


def load_workload(w: synth.Workload, extra_capacity: int = 0, with_oracle: bool = True,
                  gen_device: str = "cuda:0", extra_bytes: int = 0, extra_requests: int = 0,
                  extra_cartridges: int = 0, paged: bool = False, **kw) -> tuple:
    """Creates a Session for ``w``: registers its Cartridges, opens one request per batch entry
    (composing pool members where the workload says so) and fills the suffixes.  Returns
    (session, request handles)."""
    sess = Session(w.n_layers, w.n_q_heads, w.n_kv_heads, workload_arena_bytes(w, extra_capacity) + extra_bytes,
                   max_requests=max(w.batch, 1) + extra_requests,
                   max_cartridges=w.n_cartridges + w.batch + 1 + extra_cartridges,
                   with_oracle=with_oracle, **kw)
    cids = []
    for c in range(w.n_cartridges):
        k, v = w.cartridge_kv(c, gen_device)
        cids.append(sess.register(k, v))
        del k, v
    reqs: List[int] = []
    suffix = w.suffix_lengths()
    for b, parts in enumerate(w.request_parts()):
        if not parts:
            cart = binding.CART_NONE
        elif len(parts) == 1:
            cart = cids[parts[0]]
        else:
            cart = sess.compose([cids[p] for p in parts])
        r = sess.open(cart, int(suffix[b]) + extra_capacity, paged=paged)
        k, v = w.suffix_kv(b, int(suffix[b]), gen_device)
        sess.extend(r, k, v)
        reqs.append(r)
    return sess, reqs
