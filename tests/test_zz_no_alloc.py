"""cart_decode_attention_static -- the entry point for callers that cannot allocate device memory
(code running while an allocator pool is frozen, plug-ins that only receive tensors, early health
checks).  Its scratch is a fixed device array inside libcart.so, so the test checks that it gives what
the context-based entry point gives, twice in a row: the second call finds the first call's
leftovers in the shared scratch and must not be disturbed by them.

This file sorts last on purpose: a run that stops at the first failure has then already run every
other test."""
import numpy as np
import pytest
import torch

import oracle
from paper_2506_06266_b200 import binding, synth

import cart_harness as H

pytestmark = pytest.mark.gpu


def context_path(k, v, q):
    """Reference result from cart_decode_attention: every request gets its own one-layer Cartridge."""
    B, Hkv, n, D = k.shape
    Hq = q.shape[1]
    sess = H.Session(1, Hq, Hkv, 2 * k.numel() * 2 + (1 << 20), max_requests=B, max_cartridges=B,
                     with_oracle=False)
    try:
        reqs = []
        for b in range(B):
            c = binding.cart_register_cartridge(sess.ctx, k[b:b + 1], v[b:b + 1], n)
            reqs.append(binding.cart_request_open(sess.ctx, c, 0))
        return sess.decode(0, reqs, q)
    finally:
        sess.close()


def static_path(k, v, q):
    B, Hkv, n, D = k.shape
    Hq = q.shape[1]
    kv = torch.stack([k, v]).contiguous()
    assert kv.data_ptr() % 256 == 0
    out = torch.full_like(q, float("nan"))
    lse = torch.full((B, Hq), float("nan"), dtype=torch.float32, device=q.device)
    binding.cart_decode_attention_static(q, kv, B, Hq, Hkv, n, out, lse, device=q.device.index or 0)
    torch.cuda.synchronize(q.device)
    return out, lse


def close(a, b):
    oa, la = a
    ob, lb = b
    d = (oa.double() - ob.double())
    assert torch.isfinite(oa).all() and torch.isfinite(la).all()
    assert float(d.abs().max()) <= H.TOL_MAX_ABS
    assert float(d.norm() / ob.double().norm()) <= H.TOL_REL_FRO
    assert float((la.double() - lb.double()).abs().max()) <= H.TOL_LSE


def test_static_scratch_entry_point_matches_the_context_path_twice_in_a_row():
    H.ensure_built()
    dev = torch.device("cuda:0")
    torch.cuda.set_device(dev)
    # first call: ragged length, rows split across blocks (leaves partials and a plan in the scratch)
    k1 = synth.normal_bf16((5, 8, 2333, 128), 9001, dev)
    v1 = synth.normal_bf16((5, 8, 2333, 128), 9002, dev)
    q1 = synth.normal_bf16((5, 24, 128), 9003, dev)
    # second call: other batch, group size and length
    k2 = synth.normal_bf16((9, 8, 700, 128), 9004, dev)
    v2 = synth.normal_bf16((9, 8, 700, 128), 9005, dev)
    q2 = synth.normal_bf16((9, 32, 128), 9006, dev)
    got1 = static_path(k1, v1, q1)
    got2 = static_path(k2, v2, q2)
    close(got1, context_path(k1, v1, q1))
    close(got2, context_path(k2, v2, q2))
    # and the first problem again, after the second one has overwritten the scratch
    got1b = static_path(k1, v1, q1)
    assert torch.equal(got1[0], got1b[0]) and torch.equal(got1[1], got1b[1])


def test_static_scratch_entry_point_matches_the_cpu_oracle():
    """Directly against the float64 oracle (not only against the context path, which runs the same kernel):
    every request is one segment of n tokens per KV head."""
    H.ensure_built()
    dev = torch.device("cuda:0")
    torch.cuda.set_device(dev)
    for seed, (B, Hq, Hkv, n) in enumerate([(3, 24, 8, 1501), (7, 32, 8, 65), (2, 8, 1, 4000)]):
        k = synth.normal_bf16((B, Hkv, n, 128), 9100 + 3 * seed, dev)
        v = synth.normal_bf16((B, Hkv, n, 128), 9101 + 3 * seed, dev)
        q = synth.normal_bf16((B, Hq, 128), 9102 + 3 * seed, dev)
        kb, vb = synth.bits(k), synth.bits(v)
        ref_o, ref_l = oracle.decode_layer(synth.bits(q), [[(kb[b], vb[b])] for b in range(B)], 128 ** -0.5)
        for _ in range(2):                      # twice: the second call starts from the first one's leftovers
            out, lse = static_path(k, v, q)
            H.assert_close(out, lse, ref_o, ref_l, "static entry point, B=%d Hq=%d Hkv=%d n=%d" % (B, Hq, Hkv, n))


def test_sizes_beyond_the_fixed_scratch_are_refused():
    H.ensure_built()
    dev = torch.device("cuda:0")
    torch.cuda.set_device(dev)
    q = torch.zeros(1, 8, 128, dtype=torch.bfloat16, device=dev)
    kv = torch.zeros(2, 1, 8, 64, 128, dtype=torch.bfloat16, device=dev)
    out = torch.empty_like(q)
    with pytest.raises(binding.CartError) as ei:     # 257 requests x 8 KV heads > 2048 row groups
        binding.cart_decode_attention_static(q, kv, 257, 8, 8, 64, out)
    assert ei.value.status == binding.CART_ERR_CAPACITY
    with pytest.raises(binding.CartError) as ei:
        binding.cart_decode_attention_static(q, kv, 1, 72, 8, 64, out)
    assert ei.value.status == binding.CART_ERR_SHAPE
    with pytest.raises(binding.CartError) as ei:
        binding.cart_decode_attention_static(q, kv.data_ptr() + 16, 1, 8, 8, 64, out)
    assert ei.value.status == binding.CART_ERR_INVALID_ARG
