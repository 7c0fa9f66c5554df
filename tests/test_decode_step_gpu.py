"""GPU parity of cart_decode_step (append and attend in one launch) against the float64 CPU oracle,
and against the two separate calls it stands for."""
import pytest
import torch

from paper_2506_06266_b200 import binding, synth

import cart_harness as H

pytestmark = pytest.mark.gpu


def run_steps(w, steps, extra_capacity=None):
    sess, reqs = H.load_workload(w, extra_capacity=steps if extra_capacity is None else extra_capacity)
    try:
        for step in range(steps):
            kn, vn = w.appended_kv(step, "cuda:0")
            q = w.queries(step, "cuda:0")
            for layer in range(w.n_layers):
                out, lse = sess.decode_step(layer, reqs, kn[layer], vn[layer], q[layer])
                ro, rl = sess.oracle_decode(layer, reqs, q[layer])
                H.assert_close(out, lse, ro, rl, "%s step %d layer %d" % (w.name, step, layer))
                # the token is in the cache now: a plain decode call sees exactly the same cache
                out2, lse2 = sess.decode(layer, reqs, q[layer])
                assert torch.equal(out, out2) and torch.equal(lse, lse2)
        suffix = w.suffix_lengths()
        for b, r in enumerate(reqs):
            for layer in range(w.n_layers):
                assert binding.cart_suffix_len(sess.ctx, r, layer) == int(suffix[b]) + steps
    finally:
        sess.close()


def test_private_cartridges_growing_across_a_tile_boundary():
    # suffixes start at 61..66 tokens: the appended token lands at the end of a tile, then opens a new one
    run_steps(synth.Workload("step_priv", 501, 2, 24, 8, 6, 300, 61, 66), steps=5)


def test_requests_that_start_with_nothing_but_the_new_token():
    run_steps(synth.Workload("step_none", 502, 1, 32, 8, 5, 1, 0, 0, cartridges="none"), steps=3)


def test_cartridge_only_requests_get_their_first_suffix_token():
    run_steps(synth.Workload("step_first", 503, 2, 24, 8, 4, 200, 0, 0), steps=2)


def test_shared_cartridge_batch():
    run_steps(synth.shrink(synth.config3(), n_layers=2, batch=21, p=512), steps=3)


def test_long_rows_split_over_blocks():
    run_steps(synth.Workload("step_long", 504, 1, 32, 8, 2, 20_000, 5, 300), steps=2)


def test_many_short_requests():
    run_steps(synth.Workload("step_many", 505, 1, 24, 8, 60, 130, 1, 40), steps=2)


def test_errors_append_nothing():
    w = synth.Workload("step_err", 506, 1, 24, 8, 2, 64, 1, 1)
    sess, reqs = H.load_workload(w, extra_capacity=0)      # capacity 64, one token used
    try:
        ctx = sess.ctx
        kn, vn = w.appended_kv(0, "cuda:0")
        q = w.queries(0, "cuda:0")[0]
        out = torch.empty_like(q)
        with pytest.raises(binding.CartError) as ei:
            binding.cart_decode_step(ctx, 0, [reqs[0], reqs[0]], kn[0], vn[0], q, out)
        assert ei.value.status == binding.CART_ERR_INVALID_ARG
        with pytest.raises(binding.CartError) as ei:
            binding.cart_decode_step(ctx, 1, reqs, kn[0], vn[0], q, out)
        assert ei.value.status == binding.CART_ERR_BAD_HANDLE
        with pytest.raises(binding.CartError) as ei:
            binding.cart_decode_step(ctx, 0, reqs, kn[0], vn[0], q.data_ptr() + 2, out)
        assert ei.value.status == binding.CART_ERR_INVALID_ARG
        assert [binding.cart_suffix_len(ctx, r, 0) for r in reqs] == [1, 1]
        big = torch.zeros(63, 8, 128, dtype=torch.bfloat16, device="cuda:0")
        binding.cart_extend_kv(ctx, 0, reqs[1], big, big, 63)                  # request 1 is full now
        with pytest.raises(binding.CartError) as ei:
            binding.cart_decode_step(ctx, 0, reqs, kn[0], vn[0], q, out)
        assert ei.value.status == binding.CART_ERR_CAPACITY
        assert [binding.cart_suffix_len(ctx, r, 0) for r in reqs] == [1, 64]
        binding.cart_sync_status(ctx)
    finally:
        sess.close()
