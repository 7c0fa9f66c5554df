"""GPU parity: libcart.so (through the C ABI) against the float64 CPU oracle, element by element,
on seeded synthetic workloads shaped like the benchmark configurations but sized so the oracle
finishes in seconds, plus the degenerate cases of the method."""
import numpy as np
import pytest
import torch

from paper_2506_06266_b200 import binding, synth

import cart_harness as H

pytestmark = pytest.mark.gpu


def check_all_layers(sess, reqs, w, step=0, layers=None):
    q = w.queries(step, "cuda:0")
    worst = {"max_abs": 0.0, "rel_fro": 0.0, "lse": 0.0}
    for layer in (layers if layers is not None else range(w.n_layers)):
        r = sess.decode_and_check(layer, reqs, q[layer], "%s layer %d step %d" % (w.name, layer, step))
        for k2 in worst:
            worst[k2] = max(worst[k2], r[k2])
    return worst


def test_config1_single_layer_batch4():
    w = synth.config1()
    sess, reqs = H.load_workload(w)
    try:
        r = check_all_layers(sess, reqs, w)
        assert r["rel_fro"] < 6e-3          # bf16 output rounding alone is about 2e-3
    finally:
        sess.close()


def test_config2_shape_small_batch_with_outlier_channels():
    w = synth.shrink(synth.config2(), n_layers=3, batch=12, outlier_prob=0.01)
    assert w.outlier_mask().sum() > 0
    sess, reqs = H.load_workload(w)
    try:
        check_all_layers(sess, reqs, w)
    finally:
        sess.close()


def test_config3_shape_shared_cartridge_with_decode_appends():
    w = synth.shrink(synth.config3(), n_layers=2, batch=24)
    steps = 5
    sess, reqs = H.load_workload(w, extra_capacity=steps)
    try:
        for step in range(steps):
            kn, vn = w.appended_kv(step, "cuda:0")
            q = w.queries(step, "cuda:0")
            for layer in range(w.n_layers):
                sess.append(layer, reqs, kn[layer], vn[layer])
                if step in (0, steps - 1):
                    sess.decode_and_check(layer, reqs, q[layer], "c3 step %d layer %d" % (step, layer))
                else:
                    sess.decode(layer, reqs, q[layer])
        for b, r in enumerate(reqs):
            assert binding.cart_suffix_len(sess.ctx, r, 0) == int(w.suffix_lengths()[b]) + steps
    finally:
        sess.close()


def test_config4_shape_composed_pairs_equal_physical_concatenation():
    w = synth.shrink(synth.config4(), n_layers=2, batch=10, pool=5)
    sess, reqs = H.load_workload(w, extra_bytes=3 * (40 << 20), extra_requests=3, extra_cartridges=3)
    try:
        check_all_layers(sess, reqs, w)
        # compose(A, B) must equal one Cartridge that physically holds A || B  (Sec. 3.1, Sec. 5.4)
        parts = w.request_parts()
        q = w.queries(0, "cuda:0")
        for b in range(3):
            ka, va = w.cartridge_kv(parts[b][0], "cuda:0")
            kb, vb = w.cartridge_kv(parts[b][1], "cuda:0")
            cat = sess.register(torch.cat([ka, kb], dim=2), torch.cat([va, vb], dim=2))
            r2 = sess.open(cat, int(w.suffix_lengths()[b]))
            k, v = w.suffix_kv(b, int(w.suffix_lengths()[b]), "cuda:0")
            sess.extend(r2, k, v)
            for layer in range(w.n_layers):
                qq = q[layer][b:b + 1]
                o1, l1 = sess.decode(layer, [reqs[b]], qq)
                o2, l2 = sess.decode(layer, [r2], qq)
                # same tokens in the same order; only the tiling of the 4096 tokens may differ
                assert torch.allclose(o1.float(), o2.float(), atol=2e-3, rtol=0)
                assert torch.allclose(l1, l2, atol=1e-4, rtol=0)
    finally:
        sess.close()


def test_long_context_rows_split_over_many_blocks():
    w = synth.shrink(synth.config5_full(), n_layers=1, batch=2, p=100_000)
    sess, reqs = H.load_workload(w)
    try:
        check_all_layers(sess, reqs, w)
    finally:
        sess.close()


def test_config5_cartridge_shape_many_small_requests():
    w = synth.shrink(synth.config5_cartridge(), n_layers=1, batch=40)
    sess, reqs = H.load_workload(w)
    try:
        check_all_layers(sess, reqs, w)
    finally:
        sess.close()


@pytest.mark.parametrize("Hq,Hkv", [(8, 8), (16, 8), (24, 8), (64, 8), (8, 1), (5, 1)])
def test_group_sizes(Hq, Hkv):
    w = synth.Workload("groups", 7 + Hq, 1, Hq, Hkv, 3, 200, 1, 90)
    sess, reqs = H.load_workload(w)
    try:
        check_all_layers(sess, reqs, w)
    finally:
        sess.close()


@pytest.mark.parametrize("p,suffix", [(1, 0), (1, 1), (63, 0), (64, 0), (65, 1), (127, 130), (0, 1), (0, 64), (0, 193),
                                      (333, 15), (4096, 0)])
def test_ragged_and_degenerate_lengths(p, suffix):
    # p = 0: suffix-only request (CART_NONE); suffix = 0: Cartridge-only request
    kind = "none" if p == 0 else "private"
    w = synth.Workload("edge", 100 + p + suffix, 2, 24, 8, 3, max(p, 1), suffix, suffix, cartridges=kind)
    sess, reqs = H.load_workload(w, extra_capacity=0)
    try:
        check_all_layers(sess, reqs, w)
    finally:
        sess.close()


def test_one_token_cache_returns_its_value_exactly():
    w = synth.Workload("one", 5, 1, 24, 8, 2, 1, 1, 1, cartridges="none")
    sess, reqs = H.load_workload(w)
    try:
        q = w.queries(0, "cuda:0")[0]
        out, lse = sess.decode(0, reqs, q)
        for b in range(2):
            _, v = w.suffix_kv(b, 1, "cuda:0")          # [L][1][Hkv][D]
            expect = v[0, 0].repeat_interleave(3, dim=0)  # each KV head serves 3 query heads
            assert torch.equal(out[b], expect)
    finally:
        sess.close()


def test_composition_of_eight_parts_and_nested_compose():
    w = synth.Workload("parts", 77, 2, 16, 8, 1, 150, 9, 9, cartridges="pool", pool=8, compose=8)
    sess = H.Session(2, 16, 8, 64 << 20)
    try:
        cids = [sess.register(*w.cartridge_kv(c, "cuda:0")) for c in range(8)]
        ab = sess.compose(cids[:3])
        rest = sess.compose(cids[3:])
        full = sess.compose([ab, rest])            # nested: flattened to 8 parts
        r = sess.open(full, 9)
        k, v = w.suffix_kv(0, 9, "cuda:0")
        sess.extend(r, k, v)
        assert sess.oc.kv_tokens(0, sess.req_map[r]) == 8 * 150 + 9
        q = w.queries(0, "cuda:0")
        for layer in range(2):
            sess.decode_and_check(layer, [r], q[layer])
        with pytest.raises(binding.CartError) as ei:
            binding.cart_compose(sess.ctx, [full, cids[0]])   # nine parts
        assert ei.value.status == binding.CART_ERR_CAPACITY
    finally:
        sess.close()


def test_duplicate_requests_in_a_batch_and_null_lse():
    w = synth.Workload("dup", 9, 1, 24, 8, 2, 100, 10, 10)
    sess, reqs = H.load_workload(w, extra_requests=1)
    try:
        q = w.queries(0, "cuda:0")[0]
        batch = [reqs[0], reqs[1], reqs[0]]
        qq = torch.stack([q[0], q[1], q[0]])
        out, lse = sess.decode(0, batch, qq)
        # the two copies may be split across blocks differently: equal up to fp32 rounding of the split
        assert float((out[0].float() - out[2].float()).abs().max()) < 4e-3
        assert float((lse[0] - lse[2]).abs().max()) < 2e-4
        out2, none = sess.decode(0, batch, qq, want_lse=False)
        assert none is None and torch.equal(out, out2)
        ro, rl = sess.oracle_decode(0, batch, qq)
        H.assert_close(out, lse, ro, rl)
    finally:
        sess.close()


def test_results_are_bitwise_reproducible():
    w = synth.shrink(synth.config2(), n_layers=1, batch=20)
    sess, reqs = H.load_workload(w, with_oracle=False)
    try:
        q = w.queries(0, "cuda:0")[0]
        o1, l1 = sess.decode(0, reqs, q)
        for _ in range(3):
            o2, l2 = sess.decode(0, reqs, q)
            assert torch.equal(o1, o2) and torch.equal(l1, l2)
    finally:
        sess.close()


def test_garbage_after_a_segment_end_never_leaks_into_the_result():
    # the arena starts full of NaN bit patterns: rows past a ragged end must not reach the output
    w = synth.Workload("nan", 31, 1, 24, 8, 4, 70, 3, 50)
    sess, reqs = H.load_workload(w, extra_capacity=40, arena_fill=0x7FC0)
    try:
        check_all_layers(sess, reqs, w)
    finally:
        sess.close()


def test_arena_space_is_reused_after_release_and_close():
    sess = H.Session(1, 24, 8, 8 << 20, max_requests=4, max_cartridges=4)
    try:
        wa = synth.Workload("a", 41, 1, 24, 8, 1, 300, 5, 5)
        wb = synth.Workload("b", 42, 1, 24, 8, 1, 280, 7, 7)
        for w in (wa, wb, wa):
            c = sess.register(*w.cartridge_kv(0, "cuda:0"))
            r = sess.open(c, 10)
            sess.extend(r, *w.suffix_kv(0, int(w.suffix_lengths()[0]), "cuda:0"))
            sess.decode_and_check(0, [r], w.queries(0, "cuda:0")[0])
            with pytest.raises(binding.CartError) as ei:
                binding.cart_release_cartridge(sess.ctx, c)
            assert ei.value.status == binding.CART_ERR_IN_USE
            binding.cart_request_close(sess.ctx, r)
            binding.cart_release_cartridge(sess.ctx, c)
    finally:
        sess.close()


def test_error_paths_leave_state_untouched():
    sess = H.Session(2, 24, 8, 4 << 20, max_requests=2, max_cartridges=2)
    try:
        w = synth.Workload("e", 51, 2, 24, 8, 1, 64, 1, 1)
        k, v = w.cartridge_kv(0, "cuda:0")
        c = sess.register(k, v)
        r = sess.open(c, 64)
        q = w.queries(0, "cuda:0")[0]
        out = torch.empty_like(q)
        ctx = sess.ctx

        def status_of(fn, *a):
            with pytest.raises(binding.CartError) as ei:
                fn(*a)
            return ei.value.status

        assert status_of(binding.cart_decode_attention, ctx, 2, [r], q, out) == binding.CART_ERR_BAD_HANDLE
        assert status_of(binding.cart_decode_attention, ctx, 0, [r + 1], q, out) == binding.CART_ERR_BAD_HANDLE
        assert status_of(binding.cart_decode_attention, ctx, 0, [], q, out) == binding.CART_ERR_INVALID_ARG
        assert status_of(binding.cart_decode_attention, ctx, 0, [r], q.data_ptr() + 2, out) == binding.CART_ERR_INVALID_ARG
        assert status_of(binding.cart_decode_attention, ctx, 0, [r, r, r], q, out) == binding.CART_ERR_CAPACITY
        r_empty = sess.open(binding.CART_NONE, 64)
        assert status_of(binding.cart_decode_attention, ctx, 0, [r_empty], q, out) == binding.CART_ERR_EMPTY
        assert status_of(binding.cart_request_open, ctx, c, 8) == binding.CART_ERR_CAPACITY      # table full
        assert status_of(binding.cart_request_open, ctx, 5, 8) == binding.CART_ERR_BAD_HANDLE
        kn = torch.zeros(2, 8, 128, dtype=torch.bfloat16, device="cuda:0")
        assert status_of(binding.cart_append_kv, ctx, 0, [r, r], kn, kn) == binding.CART_ERR_INVALID_ARG
        # fill the suffix, then one more append must fail and change nothing
        big = torch.zeros(64, 8, 128, dtype=torch.bfloat16, device="cuda:0")
        binding.cart_extend_kv(ctx, 0, r, big, big, 64)
        assert status_of(binding.cart_append_kv, ctx, 0, [r_empty, r], kn, kn) == binding.CART_ERR_CAPACITY
        assert binding.cart_suffix_len(ctx, r, 0) == 64 and binding.cart_suffix_len(ctx, r_empty, 0) == 0
        assert status_of(binding.cart_extend_kv, ctx, 0, r, big, big, 1) == binding.CART_ERR_CAPACITY
        assert status_of(binding.cart_register_cartridge, ctx, k, v, 10 ** 6) == binding.CART_ERR_OOM
        c2 = sess.register(k, v)
        assert status_of(binding.cart_register_cartridge, ctx, k, v, 64) == binding.CART_ERR_CAPACITY
        assert status_of(binding.cart_release_cartridge, ctx, c) == binding.CART_ERR_IN_USE
        binding.cart_release_cartridge(ctx, c2)
        assert status_of(binding.cart_release_cartridge, ctx, c2) == binding.CART_ERR_BAD_HANDLE
        logical, private = binding.cart_kv_bytes(ctx, r)
        assert private == 64 * 4096 and logical == (2 * 64 + 64) * 4096
        binding.cart_sync_status(ctx)
    finally:
        sess.close()


def test_plan_is_rebuilt_when_lengths_or_batch_change():
    w = synth.Workload("plan", 61, 2, 24, 8, 6, 500, 1, 200)
    sess, reqs = H.load_workload(w, extra_capacity=3)
    try:
        q = w.queries(0, "cuda:0")
        sess.decode_and_check(0, reqs, q[0])
        sess.decode_and_check(1, reqs, q[1])                 # same plan, other layer
        sess.decode_and_check(0, reqs[:3], q[0][:3])         # smaller batch
        sess.decode_and_check(0, reqs[::-1], q[0].flip(0))   # other order
        kn, vn = w.appended_kv(0, "cuda:0")
        sess.append(0, reqs, kn[0], vn[0])                   # layer 0 grows, layer 1 does not
        sess.decode_and_check(0, reqs, q[0])
        sess.decode_and_check(1, reqs, q[1])
        launches = binding.cart_launch_count(sess.ctx)
        assert launches > 0
    finally:
        sess.close()


def test_cartridge_swapped_in_from_pinned_host_memory_while_others_stay():
    # hot swap: one Cartridge is released and another registered from page-locked host memory in its place
    wa = synth.Workload("swap_a", 71, 2, 24, 8, 1, 300, 4, 4)
    wb = synth.Workload("swap_b", 72, 2, 24, 8, 1, 300, 6, 6)
    sess = H.Session(2, 24, 8, 16 << 20, max_requests=4, max_cartridges=4)
    try:
        ca = sess.register(*wa.cartridge_kv(0, "cuda:0"))
        ra = sess.open(ca, 8)
        sess.extend(ra, *wa.suffix_kv(0, 4, "cuda:0"))
        kb, vb = wb.cartridge_kv(0, "cpu")
        kb_h, vb_h = kb.pin_memory(), vb.pin_memory()
        stream = torch.cuda.current_stream()
        cb = binding.cart_register_cartridge(sess.ctx, kb_h, vb_h, 300, stream)
        torch.cuda.synchronize()
        sess.cart_map[cb] = sess.oc.register(synth.bits(kb), synth.bits(vb))
        rb = sess.open(cb, 8)
        sess.extend(rb, *wb.suffix_kv(0, 6, "cuda:0"))
        q = synth.normal_bf16((2, 24, 128), 73, "cuda:0")
        for layer in range(2):
            sess.decode_and_check(layer, [ra, rb], q)
        # swap A out, a third one in (from host again), B untouched
        binding.cart_request_close(sess.ctx, ra)
        binding.cart_release_cartridge(sess.ctx, ca)
        wc = synth.Workload("swap_c", 74, 2, 24, 8, 1, 280, 3, 3)
        kc, vc = wc.cartridge_kv(0, "cpu")
        kc_h, vc_h = kc.pin_memory(), vc.pin_memory()
        cc = binding.cart_register_cartridge(sess.ctx, kc_h, vc_h, 280, stream)
        torch.cuda.synchronize()
        sess.cart_map[cc] = sess.oc.register(synth.bits(kc), synth.bits(vc))
        rc = sess.open(cc, 8)
        sess.extend(rc, *wc.suffix_kv(0, 3, "cuda:0"))
        for layer in range(2):
            sess.decode_and_check(layer, [rb, rc], q)
    finally:
        sess.close()
