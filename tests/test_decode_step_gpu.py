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


def fused_steps_on_one_plan(w, steps, check_every=1):
    """`steps` fused decode steps back to back, every call checked against the oracle; returns how many
    plans the context built over them."""
    sess, reqs = H.load_workload(w, extra_capacity=steps)
    try:
        before = binding.cart_plan_count(sess.ctx)
        for step in range(steps):
            kn, vn = w.appended_kv(step, "cuda:0")
            q = w.queries(step, "cuda:0")
            for layer in range(w.n_layers):
                out, lse = sess.decode_step(layer, reqs, kn[layer], vn[layer], q[layer])
                if step % check_every == 0 or step == steps - 1:
                    ro, rl = sess.oracle_decode(layer, reqs, q[layer])
                    H.assert_close(out, lse, ro, rl, "%s step %d layer %d" % (w.name, step, layer))
        return binding.cart_plan_count(sess.ctx) - before
    finally:
        sess.close()


def test_140_fused_steps_on_one_layer_keep_one_plan_across_two_tile_boundaries():
    # One layer, so the kernel right before a step's kernel is the previous step's, which wrote the token in
    # the tile before the new tail tile whenever a suffix length is a multiple of 64; two requests give a grid
    # well below the SM count, so consecutive kernels are resident together.  Suffixes start at 50..70 and
    # grow by 140: every request crosses two or three tile boundaries on the plan of the first step.
    w = synth.Workload("step_keep", 507, 1, 24, 8, 2, 200, 50, 70)
    assert fused_steps_on_one_plan(w, 140) == 1


def test_fused_steps_keep_one_plan_with_a_shared_cartridge_and_several_layers():
    w = synth.shrink(synth.config3(), n_layers=3, batch=9, p=400, suffix_lo=60, suffix_hi=66)
    assert fused_steps_on_one_plan(w, 70, check_every=3) == 1


def test_plan_reuse_switched_off_builds_a_plan_per_step():
    w = synth.Workload("step_replan", 508, 2, 32, 8, 3, 100, 62, 64)
    sess, reqs = H.load_workload(w, extra_capacity=4)
    try:
        binding.cart_set_plan_reuse(sess.ctx, 0)
        before = binding.cart_plan_count(sess.ctx)
        for step in range(4):
            kn, vn = w.appended_kv(step, "cuda:0")
            q = w.queries(step, "cuda:0")
            for layer in range(w.n_layers):
                out, lse = sess.decode_step(layer, reqs, kn[layer], vn[layer], q[layer])
                ro, rl = sess.oracle_decode(layer, reqs, q[layer])
                H.assert_close(out, lse, ro, rl, "step %d layer %d" % (step, layer))
        assert binding.cart_plan_count(sess.ctx) - before == 4     # one per step, shared by the layers
    finally:
        sess.close()


def test_requests_growing_by_different_amounts_get_a_new_plan():
    w = synth.Workload("step_uneven", 509, 1, 24, 8, 3, 100, 10, 12)
    sess, reqs = H.load_workload(w, extra_capacity=80)
    try:
        kn, vn = w.appended_kv(0, "cuda:0")
        q = w.queries(0, "cuda:0")
        sess.decode_step(0, reqs, kn[0], vn[0], q[0])
        n0 = binding.cart_plan_count(sess.ctx)
        sess.extend(reqs[1], *w.suffix_kv(7, 70, "cuda:0"))          # only request 1 grows, past a tile boundary
        H.assert_close(*sess.decode(0, reqs, q[0]), *sess.oracle_decode(0, reqs, q[0]), "after the uneven growth")
        assert binding.cart_plan_count(sess.ctx) == n0 + 1
    finally:
        sess.close()


def test_prefill_then_fused_steps_on_one_layer_across_a_tile_boundary():
    # The message's tokens are written by the extend kernel right before the prefill kernels, and each fused
    # step's token by the kernel right before the next step's: small grids, one layer, lengths 60 -> 127 -> 140.
    w = synth.Workload("step_prefill", 510, 1, 32, 8, 1, 256, 60, 60)
    sess = H.Session(1, 32, 8, 32 << 20, max_requests=80)
    try:
        req = sess.open(sess.register(*w.cartridge_kv(0, "cuda:0")), 60 + 67 + 13)
        sess.extend(req, *w.suffix_kv(0, 60, "cuda:0"))
        km, vm = w.suffix_kv(1, 67, "cuda:0")
        sess.extend(req, km, vm)
        qm = synth.normal_bf16((67, 32, 128), 5100, "cuda:0")
        out = torch.full_like(qm, float("nan"))
        lse = torch.full((67, 32), float("nan"), dtype=torch.float32, device="cuda:0")
        binding.cart_prefill_attention(sess.ctx, 0, req, qm, 67, out, lse)
        binding.cart_sync_status(sess.ctx)
        # the last row of the prefill is the decode result at length 127
        o1, l1 = sess.decode(0, [req], qm[-1:])
        ro, rl = sess.oracle_decode(0, [req], qm[-1:])
        H.assert_close(o1, l1, ro, rl, "decode after prefill")
        H.assert_close(out[-1:], lse[-1:], ro, rl, "last prefill row")
        for step in range(13):
            kn, vn = w.appended_kv(step, "cuda:0")
            q = w.queries(step, "cuda:0")
            o, l = sess.decode_step(0, [req], kn[0], vn[0], q[0])
            H.assert_close(o, l, *sess.oracle_decode(0, [req], q[0]), "step %d after prefill" % step)
    finally:
        sess.close()
