"""GPU parity of training-time attention over a shared trainable Cartridge (forward and backward through the C ABI)
against the float64 oracle written from the definition (oracle/train_oracle.py): conversations of ragged lengths
packed back to back, Cartridges that end inside a tile, every group size, no Cartridge at all, a layer other than
the first.  Outputs: bf16 out and fp32 lse at the decode tolerances; gradients (fp32, from bf16 tensor-core
products) within 1e-2 relative in the Frobenius norm and 2e-2 of the largest entry element by element."""
import numpy as np
import pytest
import torch

from oracle import train_oracle as TO
from paper_2506_06266_b200 import binding, synth

import cart_harness as H

pytestmark = pytest.mark.gpu
DEV = "cuda:0"

GRAD_REL = 1e-2
GRAD_MAX = 2e-2


def f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().to(torch.float64).cpu().numpy()


def rand_bf16(gen, *shape, scale=1.0):
    return (torch.randn(*shape, device=DEV, generator=gen) * scale).to(torch.bfloat16)


def run(lens, Hq, Hkv, p, layers=1, layer=0, seed=0, scale=0.0):
    gen = torch.Generator(DEV).manual_seed(1000 + seed)
    T = int(sum(lens))
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    sess = H.Session(layers, Hq, Hkv, 64 << 20, max_requests=max(T, 8), max_cartridges=4, with_oracle=False,
                     scale=scale, arena_fill=0x7FC0)
    try:
        eff_scale = scale if scale > 0 else 128 ** -0.5
        zk = rand_bf16(gen, layers, Hkv, max(p, 1), 128)[:, :, :p].contiguous()
        zv = rand_bf16(gen, layers, Hkv, max(p, 1), 128)[:, :, :p].contiguous()
        cart = binding.cart_register_cartridge(sess.ctx, zk, zv, p) if p > 0 else binding.CART_NONE
        q = rand_bf16(gen, T, Hq, 128)
        k = rand_bf16(gen, T, Hkv, 128)
        v = rand_bf16(gen, T, Hkv, 128)
        dout = rand_bf16(gen, T, Hq, 128)
        convs = []
        for c, n in enumerate(lens):
            r = binding.cart_request_open(sess.ctx, cart, n)
            a, b = int(cu[c]), int(cu[c + 1])
            binding.cart_extend_kv(sess.ctx, layer, r, k[a:b].contiguous(), v[a:b].contiguous(), n)
            convs.append(r)
        out = torch.full_like(q, float("nan"))
        lse = torch.full((T, Hq), float("nan"), dtype=torch.float32, device=DEV)
        binding.cart_train_attention_fwd(sess.ctx, layer, convs, q, out, lse)
        binding.cart_sync_status(sess.ctx)

        zk64 = f64(zk[layer]) if p > 0 else np.zeros((Hkv, 0, 128))
        zv64 = f64(zv[layer]) if p > 0 else np.zeros((Hkv, 0, 128))
        ro, rl = TO.forward(f64(q), f64(k), f64(v), zk64, zv64, cu, eff_scale)
        H.assert_close(out, lse, ro, rl, "forward")

        nan = float("nan")
        dq = torch.full((T, Hq, 128), nan, dtype=torch.float32, device=DEV)
        dk = torch.full((T, Hkv, 128), nan, dtype=torch.float32, device=DEV)
        dv = torch.full_like(dk, nan)
        dzk = torch.full((Hkv, max(p, 1), 128), nan, dtype=torch.float32, device=DEV)
        dzv = torch.full_like(dzk, nan)
        delta = torch.empty((T, Hq), dtype=torch.float32, device=DEV)
        binding.cart_train_attention_bwd(sess.ctx, layer, convs, q, out, lse, dout, delta, dq, dk, dv,
                                         dzk if p > 0 else None, dzv if p > 0 else None)
        binding.cart_sync_status(sess.ctx)
        # the oracle differentiates the exact forward; the kernel was given the forward's rounded out and lse
        g = TO.backward(f64(q), f64(k), f64(v), zk64, zv64, cu, eff_scale, f64(dout))
        got = {"dq": dq, "dk": dk, "dv": dv}
        if p > 0:
            got["dzk"], got["dzv"] = dzk[:, :p], dzv[:, :p]
        for name, t in got.items():
            a, ref = f64(t), g[name]
            assert np.all(np.isfinite(a)), name + ": non-finite gradient"
            rel = np.linalg.norm(a - ref) / max(np.linalg.norm(ref), 1e-300)
            worst = np.max(np.abs(a - ref)) / max(np.max(np.abs(ref)), 1e-300)
            assert rel <= GRAD_REL, "%s: relative (Frobenius) error %.3e" % (name, rel)
            assert worst <= GRAD_MAX, "%s: largest error %.3e of the largest entry" % (name, worst)
        # a decode plan still works after the training calls took a buffer of the plan ring
        qd = rand_bf16(gen, len(convs), Hq, 128)
        od = torch.empty_like(qd)
        binding.cart_decode_attention(sess.ctx, layer, convs, qd, od, None)
        binding.cart_sync_status(sess.ctx)
        assert torch.isfinite(od.float()).all()
    finally:
        sess.close()


def test_ragged_conversations_over_a_cartridge_that_ends_inside_a_tile():
    run([5, 1, 70, 130], 32, 8, 300, seed=1)


def test_group_of_three_heads_per_kv_head():
    # 128 / 3 is not whole: a row tile holds 42 tokens and two rows that no token owns
    run([40, 100, 3], 24, 8, 128, seed=2)


def test_conversations_without_a_cartridge():
    run([129, 31], 16, 8, 0, seed=3)


def test_one_kv_head_with_eight_query_heads_and_a_later_layer():
    run([33, 64, 17], 8, 1, 260, layers=2, layer=1, seed=4)


def test_multi_head_attention_group_of_one():
    run([150, 20], 4, 4, 140, seed=5, scale=0.11)


def test_many_short_conversations_share_a_long_cartridge():
    rng = np.random.default_rng(6)
    run([int(x) for x in rng.integers(8, 48, size=24)], 32, 8, 1024, seed=6)


def test_errors():
    sess = H.Session(1, 8, 2, 8 << 20, max_requests=16, max_cartridges=4, with_oracle=False)
    try:
        z = torch.zeros(1, 2, 64, 128, dtype=torch.bfloat16, device=DEV)
        c1 = binding.cart_register_cartridge(sess.ctx, z, z, 64)
        c2 = binding.cart_register_cartridge(sess.ctx, z, z, 64)
        kv = torch.zeros(4, 2, 128, dtype=torch.bfloat16, device=DEV)
        r1 = binding.cart_request_open(sess.ctx, c1, 64)
        r2 = binding.cart_request_open(sess.ctx, c2, 64)
        r3 = binding.cart_request_open_paged(sess.ctx, c1, 64)
        r4 = binding.cart_request_open(sess.ctx, c1, 64)
        for r in (r1, r2, r3):
            binding.cart_extend_kv(sess.ctx, 0, r, kv, kv, 4)
        q = torch.zeros(32, 8, 128, dtype=torch.bfloat16, device=DEV)
        out = torch.zeros_like(q)
        lse = torch.zeros(32, 8, dtype=torch.float32, device=DEV)
        for convs, status in [([r1, r2], binding.CART_ERR_INVALID_ARG),      # different Cartridges
                              ([r1, r3], binding.CART_ERR_INVALID_ARG),      # a paged suffix
                              ([r1, r4], binding.CART_ERR_EMPTY),            # a conversation without tokens
                              ([r1, r1], binding.CART_ERR_INVALID_ARG),      # twice
                              ([r1, 99], binding.CART_ERR_BAD_HANDLE)]:
            with pytest.raises(binding.CartError) as ei:
                binding.cart_train_attention_fwd(sess.ctx, 0, convs, q, out, lse)
            assert ei.value.status == status
        with pytest.raises(binding.CartError) as ei:
            binding.cart_train_attention_fwd(sess.ctx, 0, [r1], q, out, None)
        assert ei.value.status == binding.CART_ERR_INVALID_ARG
        binding.cart_sync_status(sess.ctx)
    finally:
        sess.close()
