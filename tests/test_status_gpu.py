"""cart_sync_status and the device status word.  Every device-side wait of the kernels is bounded; a wait that
runs out sets a bit in a status word at the start of the arena's scratch, which cart_sync_status reports as
CART_ERR_TIMEOUT and clears together with the arrival tickets a block that gave up may have left behind.  No
kernel is made to wait here: the test writes the word itself with a plain host-to-device copy."""
import pytest
import torch

from paper_2506_06266_b200 import binding, synth

import cart_harness as H

pytestmark = pytest.mark.gpu

STATUS_OFFSET = 0      # the status word is the first word of the arena
TICKETS_OFFSET = 256   # arrival tickets follow it, one 32-bit counter per split row group


def poke(arena: torch.Tensor, offset: int, value: int) -> None:
    host = torch.tensor(list(int(value).to_bytes(4, "little")), dtype=torch.uint8)
    arena[offset:offset + 4].copy_(host)          # cudaMemcpy host -> device, no kernel
    torch.cuda.synchronize(arena.device)


def peek(arena: torch.Tensor, offset: int) -> int:
    return int.from_bytes(bytes(arena[offset:offset + 4].cpu().tolist()), "little")


def test_a_set_status_word_is_reported_as_a_timeout_then_cleared_and_decoding_goes_on():
    w = synth.Workload("status", 901, 1, 24, 8, 3, 700, 5, 90)     # rows long enough to be split over blocks
    sess, reqs = H.load_workload(w)
    try:
        q = w.queries(0, "cuda:0")[0]
        sess.decode_and_check(0, reqs, q, "before")
        assert peek(sess.arena, STATUS_OFFSET) == 0
        poke(sess.arena, STATUS_OFFSET, 2)            # "a consumer warp's wait ran out"
        poke(sess.arena, TICKETS_OFFSET, 1)           # a ticket taken by a block that then gave up
        poke(sess.arena, TICKETS_OFFSET + 8, 3)
        with pytest.raises(binding.CartError) as ei:
            binding.cart_sync_status(sess.ctx)
        assert ei.value.status == binding.CART_ERR_TIMEOUT
        assert "0x2" in str(ei.value)
        assert peek(sess.arena, STATUS_OFFSET) == 0
        assert peek(sess.arena, TICKETS_OFFSET) == 0 and peek(sess.arena, TICKETS_OFFSET + 8) == 0
        binding.cart_sync_status(sess.ctx)            # reported once
        sess.decode_and_check(0, reqs, q, "after")    # stale tickets would have corrupted the merges
    finally:
        sess.close()
