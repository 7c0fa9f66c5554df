"""Loads a synthetic workload into a libcart context and steps it, for the benchmark and the
full-size tests.  Orchestration only: every arithmetic step runs inside libcart.so.

It can keep host copies of the raw bf16 bits of chosen (layer, request) KV blocks while loading, so
that a caller may hand exactly the same inputs to a checker afterwards; it never imports one.
"""
from __future__ import annotations

from typing import Dict, Iterable, List, Optional, Sequence, Tuple

import numpy as np
import torch

from . import binding, buildlib, synth


def arena_bytes_for(w: synth.Workload, extra_capacity: int, paged: bool = False) -> int:
    per_tok = w.n_layers * w.kv_bytes_per_token_layer()
    # (a paged request may hold one page of room more than it needs: pages are taken a plan's lifetime ahead)
    caps = [-(-(int(s) + extra_capacity) // 64) * 64 + (128 if paged else 0) for s in w.suffix_lengths()]
    return (w.n_cartridges * w.p + sum(caps)) * per_tok


class LoadedWorkload:
    """A workload resident on one GPU: arena, context, Cartridge and request handles.

    keep_layers / keep_requests: layers and batch indices whose KV bits are also copied to the host
    while loading (``host_segments``), in cache order [Cartridge part(s)..., suffix].
    paged: the requests' suffixes live in pages of 64 tokens taken as they grow, not in one buffer each.
    """

    def __init__(self, w: synth.Workload, device: torch.device, extra_capacity: int = 0,
                 keep_layers: Sequence[int] = (), keep_requests: Optional[Sequence[int]] = None,
                 stream: Optional[torch.cuda.Stream] = None, paged: bool = False):
        buildlib.build()
        binding.load_library()
        self.w = w
        self.dev = torch.device(device)
        self.stream = stream
        self.keep_layers = list(keep_layers)
        self.keep_requests = list(range(w.batch)) if keep_requests is None else list(keep_requests)
        cfg = binding.make_config(w.n_layers, w.n_q_heads, w.n_kv_heads, max(w.batch, 1),
                                  w.n_cartridges + w.batch + 1, device=self.dev.index or 0,
                                  softmax_scale=w.scale)
        scratch = binding.cart_scratch_bytes(cfg)
        total = scratch + arena_bytes_for(w, extra_capacity, paged) + 4096
        self.arena = torch.empty(total, dtype=torch.uint8, device=self.dev)
        cfg.arena, cfg.arena_bytes = self.arena.data_ptr(), total
        self.cfg = cfg
        self.ctx = binding.cart_create(cfg)
        self.suffix = w.suffix_lengths()
        self.parts = w.request_parts()
        self.host_cart: Dict[Tuple[int, int], Tuple[np.ndarray, np.ndarray]] = {}
        self.host_suffix: Dict[Tuple[int, int], Tuple[np.ndarray, np.ndarray]] = {}
        kept_carts = {c for b in self.keep_requests for c in self.parts[b]} if self.keep_layers else set()

        self.cart_ids: List[int] = []
        for c in range(w.n_cartridges):
            k, v = w.cartridge_kv(c, self.dev)
            self.cart_ids.append(binding.cart_register_cartridge(self.ctx, k, v, w.p, stream))
            if c in kept_carts:
                for layer in self.keep_layers:
                    self.host_cart[(layer, c)] = (synth.bits(k[layer]), synth.bits(v[layer]))
            torch.cuda.synchronize(self.dev)
            del k, v
        self.reqs: List[int] = []
        self.composed: List[int] = []
        for b, parts in enumerate(self.parts):
            if not parts:
                cart = binding.CART_NONE
            elif len(parts) == 1:
                cart = self.cart_ids[parts[0]]
            else:
                cart = binding.cart_compose(self.ctx, [self.cart_ids[p] for p in parts])
                self.composed.append(cart)
            if paged:
                r = binding.cart_request_open_paged(self.ctx, cart, 0)
            else:
                r = binding.cart_request_open(self.ctx, cart, int(self.suffix[b]) + extra_capacity)
            n = int(self.suffix[b])
            if n > 0:
                k, v = w.suffix_kv(b, n, self.dev)      # [L][T][Hkv][D]
                for layer in range(w.n_layers):
                    binding.cart_extend_kv(self.ctx, layer, r, k[layer], v[layer], n, stream)
                if b in self.keep_requests:
                    for layer in self.keep_layers:
                        self.host_suffix[(layer, b)] = (
                            np.ascontiguousarray(np.transpose(synth.bits(k[layer]), (1, 0, 2))),
                            np.ascontiguousarray(np.transpose(synth.bits(v[layer]), (1, 0, 2))))
                torch.cuda.synchronize(self.dev)
            self.reqs.append(r)
        self.req_list = binding.ReqList(self.reqs)
        self.appended = 0   # decode steps taken so far (tokens appended per request and layer)

    # ---------------------------------------------------------------------------------------
    def host_segments(self, layer: int, b: int) -> List[Tuple[np.ndarray, np.ndarray]]:
        """Kept bits of request b's cache in `layer` as loaded (before any decode append)."""
        segs = [self.host_cart[(layer, c)] for c in self.parts[b]]
        if (layer, b) in self.host_suffix:
            segs.append(self.host_suffix[(layer, b)])
        return segs

    def kv_tokens(self) -> np.ndarray:
        """KV tokens per request right now (same in every layer between steps)."""
        return self.w.kv_tokens() + self.appended

    def algorithmic_bytes_per_layer(self) -> int:
        """K/V bytes every request must read once per layer, plus q, out and lse traffic."""
        w = self.w
        kv = int(self.kv_tokens().sum()) * w.kv_bytes_per_token_layer()
        io = w.batch * w.n_q_heads * (w.head_dim * 2 * 2 + 4)
        return kv + io

    def unique_bytes_per_layer(self) -> int:
        """What the method itself has to read per layer: every stored Cartridge the batch attends to once,
        however many requests share it, every request's own suffix, plus q, out and lse traffic."""
        w = self.w
        carts = {c for parts in self.parts for c in parts}
        suffix_tokens = int(self.suffix.sum()) + self.appended * w.batch
        kv = (len(carts) * w.p + suffix_tokens) * w.kv_bytes_per_token_layer()
        io = w.batch * w.n_q_heads * (w.head_dim * 2 * 2 + 4)
        return kv + io

    def shared_flops_per_layer(self, min_readers: int = 4, tile: int = 128) -> int:
        """Floating-point operations of the two dense products (q K^T and P V) over the full tiles of the
        Cartridges that at least `min_readers` requests of the batch share: the tensor-core kernel's work."""
        w = self.w
        readers: Dict[int, int] = {}
        for parts in self.parts:
            for c in parts:
                readers[c] = readers.get(c, 0) + 1
        full = w.p // tile * tile
        return sum(4 * r * w.n_q_heads * w.head_dim * full for r in readers.values() if r >= min_readers and full)

    def step(self, q: torch.Tensor, k_new: torch.Tensor, v_new: torch.Tensor, out: torch.Tensor,
             lse: Optional[torch.Tensor], layers: Optional[Iterable[int]] = None, fused: bool = True) -> None:
        """One decode step: per layer, append every request's new token, then attend -- in one call
        (cart_decode_step) or, with fused=False, as cart_append_kv followed by cart_decode_attention.
        q, out: [L][B][Hq][D]; k_new, v_new: [L][B][Hkv][D]; lse: [L][B][Hq] or None."""
        ctx, rl, s = self.ctx, self.req_list, self.stream
        # (addresses instead of per-layer tensor views: slicing five tensors costs more host time than a small
        #  batch's kernel takes)
        qp, op, kp, vp = q.data_ptr(), out.data_ptr(), k_new.data_ptr(), v_new.data_ptr()
        qs, ks = q.stride(0) * q.element_size(), k_new.stride(0) * k_new.element_size()
        lp = 0 if lse is None else lse.data_ptr()
        lstride = 0 if lse is None else lse.stride(0) * lse.element_size()
        for layer in (range(self.w.n_layers) if layers is None else layers):
            ls = None if lse is None else lp + layer * lstride
            if fused:
                binding.cart_decode_step(ctx, layer, rl, kp + layer * ks, vp + layer * ks, qp + layer * qs,
                                         op + layer * qs, ls, s)
            else:
                binding.cart_append_kv(ctx, layer, rl, kp + layer * ks, vp + layer * ks, s)
                binding.cart_decode_attention(ctx, layer, rl, qp + layer * qs, op + layer * qs, ls, s)
        self.appended += 1

    def close(self) -> None:
        if self.ctx:
            binding.cart_destroy(self.ctx)
            self.ctx = 0
        self.arena = None
