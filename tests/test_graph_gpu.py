"""GPU parity of the recordable decode loop (cart_graph_begin / cart_graph_step / cart_graph_end): one step over all
layers is captured into a CUDA graph once and replayed; every replay appends a token per request and layer and
attends to it (Sec. 2.3), with nothing but the contents of the input buffers changing between replays.  Every
replay is compared with the float64 oracle on the grown caches."""
import pytest
import torch

from paper_2506_06266_b200 import binding, synth

import cart_harness as H

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def run_loop(w, steps, paged=False, capture=True, max_steps=None):
    max_steps = steps if max_steps is None else max_steps
    sess, reqs = H.load_workload(w, extra_capacity=max_steps, paged=paged)
    try:
        L, B = w.n_layers, w.batch
        kn = torch.zeros(L, B, w.n_kv_heads, 128, dtype=torch.bfloat16, device=DEV)
        vn = torch.zeros_like(kn)
        q = torch.zeros(L, B, w.n_q_heads, 128, dtype=torch.bfloat16, device=DEV)
        out = torch.full_like(q, float("nan"))
        lse = torch.full((L, B, w.n_q_heads), float("nan"), dtype=torch.float32, device=DEV)
        stream = torch.cuda.Stream(device=DEV)
        launches_before = binding.cart_launch_count(sess.ctx)
        plans_before = binding.cart_plan_count(sess.ctx)
        with torch.cuda.stream(stream):
            binding.cart_graph_begin(sess.ctx, reqs, max_steps, stream)

            def one_step():
                for layer in range(L):
                    binding.cart_graph_step(sess.ctx, layer, kn[layer], vn[layer], q[layer], out[layer], lse[layer], stream)

            graph = None
            if capture:
                stream.synchronize()
                graph = torch.cuda.CUDAGraph()
                with torch.cuda.graph(graph, stream=stream):
                    one_step()
        launches_per_step = binding.cart_launch_count(sess.ctx) - launches_before if capture else None
        for step in range(steps):
            k_s, v_s = w.appended_kv(step, DEV)
            q_s = w.queries(step, DEV)
            with torch.cuda.stream(stream):
                kn.copy_(k_s)
                vn.copy_(v_s)
                q.copy_(q_s)
                out.fill_(float("nan"))
                if capture:
                    graph.replay()
                else:
                    one_step()
            stream.synchronize()
            for layer in range(L):
                sess.oc.append(layer, [sess.req_map[r] for r in reqs], synth.bits(k_s[layer]), synth.bits(v_s[layer]))
                ro, rl = sess.oracle_decode(layer, reqs, q_s[layer])
                H.assert_close(out[layer], lse[layer], ro, rl, "%s step %d layer %d" % (w.name, step, layer))
        binding.cart_sync_status(sess.ctx)
        # one plan for the whole loop; a captured step launches nothing new when it is replayed
        assert binding.cart_plan_count(sess.ctx) == plans_before + 1
        if capture:
            assert binding.cart_launch_count(sess.ctx) == launches_before + launches_per_step
        binding.cart_graph_end(sess.ctx, steps)
        suffix = w.suffix_lengths()
        for b, r in enumerate(reqs):
            for layer in range(L):
                assert binding.cart_suffix_len(sess.ctx, r, layer) == int(suffix[b]) + steps
        # the ordinary calls carry on from the grown caches
        q1 = w.queries(steps, DEV)
        sess.decode_and_check(0, reqs, q1[0], "after the loop")
    finally:
        sess.close()


def test_replayed_step_grows_private_caches_across_a_tile_boundary():
    # suffixes start at 60..66 tokens: within 8 steps the appended token ends a tile, then opens the next one
    run_loop(synth.Workload("graph_priv", 511, 3, 24, 8, 6, 300, 60, 66), steps=8)


def test_replayed_step_over_a_shared_cartridge():
    run_loop(synth.shrink(synth.config3(), n_layers=2, batch=21, p=512, suffix_lo=1, suffix_hi=140), steps=4)


def test_replayed_step_with_paged_suffixes_that_take_their_pages_at_the_start():
    run_loop(synth.Workload("graph_paged", 512, 2, 32, 8, 5, 200, 50, 70), steps=70, paged=True)


def test_requests_without_a_cartridge_and_without_tokens():
    run_loop(synth.Workload("graph_none", 513, 1, 32, 8, 4, 1, 0, 0, cartridges="none"), steps=3)


def test_the_same_calls_without_a_capture():
    run_loop(synth.Workload("graph_plain", 514, 2, 24, 8, 3, 130, 5, 40), steps=3, capture=False, max_steps=10)


def test_errors():
    w = synth.Workload("graph_err", 515, 2, 24, 8, 2, 64, 3, 3)
    sess, reqs = H.load_workload(w, extra_capacity=4)
    try:
        z = torch.zeros(2, 24, 128, dtype=torch.bfloat16, device=DEV)
        kv = torch.zeros(2, 8, 128, dtype=torch.bfloat16, device=DEV)
        with pytest.raises(binding.CartError) as ei:
            binding.cart_graph_step(sess.ctx, 0, kv, kv, z, z)                  # no loop open
        assert ei.value.status == binding.CART_ERR_INVALID_ARG
        for bad, status in [((reqs, 62), binding.CART_ERR_CAPACITY),            # capacity is a whole tile: 3 + 61 fit
                            ((reqs, 100000), binding.CART_ERR_CAPACITY),        # more than a kept plan covers
                            (([reqs[0], reqs[0]], 1), binding.CART_ERR_INVALID_ARG),
                            (([reqs[0], 77], 1), binding.CART_ERR_BAD_HANDLE),
                            ((reqs, 0), binding.CART_ERR_INVALID_ARG)]:
            with pytest.raises(binding.CartError) as ei:
                binding.cart_graph_begin(sess.ctx, *bad)
            assert ei.value.status == status
        # layers of unequal length cannot share one plan
        binding.cart_extend_kv(sess.ctx, 1, reqs[0], kv[:1], kv[:1], 1)
        with pytest.raises(binding.CartError) as ei:
            binding.cart_graph_begin(sess.ctx, reqs, 2)
        assert ei.value.status == binding.CART_ERR_INVALID_ARG
        binding.cart_extend_kv(sess.ctx, 0, reqs[0], kv[:1], kv[:1], 1)
        binding.cart_graph_begin(sess.ctx, reqs, 60)
        with pytest.raises(binding.CartError) as ei:
            binding.cart_graph_begin(sess.ctx, reqs, 2)                         # already open
        assert ei.value.status == binding.CART_ERR_IN_USE
        with pytest.raises(binding.CartError) as ei:
            binding.cart_graph_step(sess.ctx, 2, kv, kv, z, z)
        assert ei.value.status == binding.CART_ERR_BAD_HANDLE
        # another attention call takes the loop's plan away
        binding.cart_prefill_attention(sess.ctx, 0, reqs[1], z, 2, torch.empty_like(z))
        binding.cart_decode_attention(sess.ctx, 0, [reqs[1]], z[:1], torch.empty_like(z[:1]))
        with pytest.raises(binding.CartError) as ei:
            binding.cart_graph_step(sess.ctx, 0, kv, kv, z, z)
        assert ei.value.status == binding.CART_ERR_INVALID_ARG
        with pytest.raises(binding.CartError) as ei:
            binding.cart_graph_end(sess.ctx, 61)                                # more steps than the loop was opened for
        assert ei.value.status == binding.CART_ERR_INVALID_ARG
        binding.cart_graph_end(sess.ctx, 0)
        binding.cart_sync_status(sess.ctx)
    finally:
        sess.close()
