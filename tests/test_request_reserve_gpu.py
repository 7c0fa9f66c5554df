"""GPU test of cart_request_reserve: a request that outgrows the suffix capacity it was opened with is moved to a
larger buffer, keeps every token it had in every layer, and decodes like before; its neighbours are untouched."""
import pytest
import torch

from paper_2506_06266_b200 import binding, synth

import cart_harness as H

pytestmark = pytest.mark.gpu


def check_all_layers(sess, reqs, w, seed, what):
    for layer in range(w.n_layers):
        q = synth.normal_bf16((len(reqs), w.n_q_heads, 128), seed + layer, "cuda:0")
        sess.decode_and_check(layer, reqs, q, "%s, layer %d" % (what, layer))


def test_a_request_grows_past_its_first_capacity_and_keeps_its_tokens():
    w = synth.Workload("grow", 901, 2, 32, 8, 2, 300, 50, 50)
    sess = H.Session(2, 32, 8, 48 << 20, max_requests=4)
    try:
        cart = sess.register(*w.cartridge_kv(0, "cuda:0"))
        a = sess.open(cart, 64)
        b = sess.open(cart, 200)
        sess.extend(a, *w.suffix_kv(0, 50, "cuda:0"))
        sess.extend(b, *w.suffix_kv(1, 120, "cuda:0"))
        check_all_layers(sess, [a, b], w, 910, "before")

        # a is full after 64 tokens: a longer message does not fit
        k_more, v_more = w.suffix_kv(2, 200, "cuda:0")
        with pytest.raises(binding.CartError) as ei:
            binding.cart_extend_kv(sess.ctx, 0, a, k_more[0], v_more[0], 200)
        assert ei.value.status == binding.CART_ERR_CAPACITY

        binding.cart_request_reserve(sess.ctx, a, 300)
        check_all_layers(sess, [a, b], w, 920, "moved, nothing added")       # the 50 old tokens came along
        sess.extend(a, k_more, v_more)
        assert binding.cart_suffix_len(sess.ctx, a, 1) == 250
        check_all_layers(sess, [a, b], w, 930, "moved and extended")

        # decode steps with the fused append, layers of unequal length (layer 0 runs ahead)
        for step in range(3):
            for layer in range(w.n_layers if step < 2 else 1):
                kn = synth.normal_bf16((2, 8, 128), 940 + 10 * step + layer, "cuda:0")
                vn = synth.normal_bf16((2, 8, 128), 945 + 10 * step + layer, "cuda:0")
                q = synth.normal_bf16((2, 32, 128), 950 + 10 * step + layer, "cuda:0")
                out, lse = sess.decode_step(layer, [a, b], kn, vn, q)
                ro, rl = sess.oracle_decode(layer, [a, b], q)
                H.assert_close(out, lse, ro, rl, "step %d layer %d" % (step, layer))
        binding.cart_request_reserve(sess.ctx, a, 600)                       # again, with unequal layer lengths
        binding.cart_request_reserve(sess.ctx, b, 129)                       # not above its capacity: nothing happens
        check_all_layers(sess, [b, a], w, 960, "moved twice")
    finally:
        sess.close()


def test_reserve_errors_leave_the_request_as_it_was():
    w = synth.Workload("grow_e", 971, 1, 8, 8, 1, 64, 10, 10)
    sess = H.Session(1, 8, 8, 4 << 20, max_requests=2)
    try:
        r = sess.open(binding.CART_NONE, 64)
        sess.extend(r, *w.suffix_kv(0, 10, "cuda:0"))
        for req, cap, status in [(r, 1 << 22, binding.CART_ERR_OOM), (r, -1, binding.CART_ERR_INVALID_ARG),
                                 (r + 1, 128, binding.CART_ERR_BAD_HANDLE)]:
            with pytest.raises(binding.CartError) as ei:
                binding.cart_request_reserve(sess.ctx, req, cap)
            assert ei.value.status == status
        check_all_layers(sess, [r], w, 980, "after refused reserves")
        # an empty request can grow too (nothing to copy)
        e = sess.open(binding.CART_NONE, 0)
        binding.cart_request_reserve(sess.ctx, e, 70)
        sess.extend(e, *w.suffix_kv(1, 70, "cuda:0"))
        check_all_layers(sess, [r, e], w, 990, "grown from nothing")
    finally:
        sess.close()
