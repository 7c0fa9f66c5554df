"""Host planner with shared segments: every KV token of every (request, KV head) is covered exactly
once -- by a stream item or by a shared unit that lists the request among its readers -- the partial
slots of a row group are contiguous and complete, and both kernels' blocks are balanced."""
import numpy as np
import pytest

from paper_2506_06266_b200 import binding, buildlib, synth

B_, E_, D_ = binding.CART_ITEM_BEGIN, binding.CART_ITEM_END, binding.CART_ITEM_DIRECT
LAYERS = 4


@pytest.fixture(scope="module", autouse=True)
def _built():
    buildlib.build()


class Arena:
    """Hands out fake row ranges for stored segments."""

    def __init__(self, n_kv_heads):
        self.row = 1000
        self.Hkv = n_kv_heads

    def store(self, n, cap_pad=0):
        hs = n + cap_pad
        k = self.row
        self.row += LAYERS * self.Hkv * hs
        v = self.row
        self.row += LAYERS * self.Hkv * hs
        return (k, v, hs, self.Hkv * hs, n)


def check(segs, Hkv, G, n_cta, tile=64, share_min=4, share_tile=128, slots_cap=1 << 20, piece_cost=0,
          unit_cost=0, side_by_side=0):
    plan = binding.cart_plan_build_shared(segs, Hkv, G, n_cta, tile, share_min, share_tile, slots_cap, piece_cost,
                                          unit_cost, side_by_side)
    if plan["n_shared_ctas"]:
        # side by side: the two kernels' blocks fit on the device together
        assert side_by_side and plan["units"] and plan["items"]
        assert plan["n_unit_cta_used"] <= plan["n_shared_ctas"] < n_cta
        assert plan["n_cta_used"] <= n_cta - plan["n_shared_ctas"]
        if side_by_side > 1:
            assert plan["n_shared_ctas"] == min(side_by_side, n_cta - 1)
    items, cta_begin, units = plan["items"], plan["cta_begin"], plan["units"]
    R = 128 // G

    # tokens[(request, head)] = list of (k_row of token, v_row of token) covered, in any order
    cover = {}

    def add(rg, k0, v0, n):
        cover.setdefault(rg, []).extend((k0 + j, v0 + j) for j in range(n))

    # ---- stream items ---------------------------------------------------------------------------
    pieces = {}
    per_cta = []
    per_cta_pieces = []
    for c in range(n_cta):
        tiles, open_rg = 0, None
        for it in items[cta_begin[c]:cta_begin[c + 1]]:
            assert it.n_tok > 0
            if it.flags & B_:
                assert open_rg is None
                open_rg = it.row_group
            assert open_rg == it.row_group
            add(it.row_group, it.k_row, it.v_row, it.n_tok)
            tiles += -(-it.n_tok // tile)
            if it.flags & E_:
                pieces.setdefault(it.row_group, []).append((bool(it.flags & D_), it.slot, it.merge))
                open_rg = None
        assert open_rg is None
        per_cta.append(tiles)
        per_cta_pieces.append(sum(1 for it in items[cta_begin[c]:cta_begin[c + 1]] if it.flags & E_))
    used = plan["n_cta_used"]
    assert sum(per_cta) == plan["total_tiles"] and all(t == 0 for t in per_cta[used:])
    if used and piece_cost == 0:
        assert max(per_cta[:used]) - min(per_cta[:used]) <= 1 and min(per_cta[:used]) >= 1
    elif used and used == len(pieces) and all(len(v) == 1 for v in pieces.values()) and \
            all(n == 1 for n in per_cta_pieces[:used]):
        # a small batch: every row group has a block of its own and is streamed whole (no cut, no stream-side merge),
        # which the planner only does when the blocks stay short
        assert max(per_cta[:used]) <= 24 and sum(per_cta) <= 4 * n_cta and min(per_cta[:used]) >= 1
    elif used:
        # balanced by weight = tiles + piece_cost * pieces: no block is more than one piece and one tile
        # above the even share (the last block takes what is left and may be lighter)
        weight = [t + piece_cost * n for t, n in zip(per_cta[:used], per_cta_pieces[:used])]
        assert min(per_cta[:used]) >= 1
        assert max(weight) <= -(-sum(weight) // used) + piece_cost + 1
    assert cta_begin[n_cta] == len(items)

    # ---- shared units -----------------------------------------------------------------------------
    ucb = plan["unit_cta_begin"]
    uused = plan["n_unit_cta_used"]
    per_ucta = []
    per_ucta_units = []
    shared_slots = {}   # row group -> list of slots its shared chunks write
    for c in range(n_cta):
        t = 0
        for u in units[ucb[c]:ucb[c + 1]]:
            assert u.n_tiles > 0 and 1 <= u.n_readers <= R and u.kv_head < Hkv
            t += u.n_tiles
            for i in range(u.n_readers):
                e = u.reader_begin + i
                b = plan["readers"][e]
                rg = b * Hkv + u.kv_head
                add(rg, u.k_row, u.v_row, u.n_tiles * share_tile)
                shared_slots.setdefault(rg, []).append(
                    (plan["reader_slot"][e][u.kv_head] + u.chunk, plan["reader_merge"][e][u.kv_head]))
        per_ucta.append(t)
        per_ucta_units.append(ucb[c + 1] - ucb[c])
    assert sum(per_ucta) == plan["shared_tiles"] and all(t == 0 for t in per_ucta[uused:])
    if uused and unit_cost == 0:
        assert max(per_ucta[:uused]) - min(per_ucta[:uused]) <= 1 and min(per_ucta[:uused]) >= 1
    elif uused:
        weight = [t + unit_cost * n for t, n in zip(per_ucta[:uused], per_ucta_units[:uused])]
        assert min(per_ucta[:uused]) >= 1
        assert max(weight) <= -(-sum(weight) // uused) + unit_cost + 1
    assert ucb[n_cta] == len(units)

    # ---- coverage: exactly the tokens of the request's segments, each once ---------------------------
    for b, r in enumerate(segs):
        for g in range(Hkv):
            want = []
            for (k, v, hs, ls, n) in r:
                want += [(k + g * hs + j, v + g * hs + j) for j in range(n)]
            assert sorted(cover.get(b * Hkv + g, [])) == sorted(want), (b, g)

    # ---- slots and merges ----------------------------------------------------------------------------
    merges = plan["merges"]
    seen = []
    for b in range(len(segs)):
        for g in range(Hkv):
            rg = b * Hkv + g
            ps = pieces.get(rg, [])
            sh = shared_slots.get(rg, [])
            if not sh and len(ps) == 1 and ps[0][0]:
                continue                                   # written directly, no partial
            assert all(not d for d, _, _ in ps)
            ids = {m for _, _, m in ps} | {m for _, m in sh}
            assert len(ids) == 1
            mi = merges[ids.pop()]
            assert mi.row_group == rg
            slots = sorted([s for s, _ in sh] + [s for _, s, _ in ps])
            assert slots == list(range(mi.slot_begin, mi.slot_end))
            # shared chunks come first, stream pieces after
            assert sorted(s for s, _ in sh) == slots[:len(sh)]
            seen += slots
    assert sorted(seen) == list(range(plan["n_slots"]))
    assert plan["n_slots"] <= slots_cap
    return plan


def test_one_cartridge_shared_by_all_requests():
    a = Arena(8)
    cart = a.store(4096)
    segs = [[cart, a.store(int(n), cap_pad=9)] for n in np.random.default_rng(3).integers(1, 1025, size=128)]
    plan = check(segs, 8, 4, 148)
    assert plan["shared_tiles"] == 8 * 4 * 32 and plan["n_unit_cta_used"] == 148
    assert len(plan["readers"]) == 128 and plan["readers"] == list(range(128))
    # the Cartridge has left the stream entirely (4096 is a multiple of 128)
    assert plan["total_tiles"] == 8 * sum(-(-s[1][4] // 64) for s in segs)


def test_composed_pairs_from_a_pool_with_ragged_lengths():
    a = Arena(2)
    pool = [a.store(n) for n in (700, 129, 127, 1000, 385)]
    rng = np.random.default_rng(5)
    segs = []
    for _ in range(23):
        i, j = rng.choice(5, 2, replace=False)
        segs.append([pool[i], pool[j], a.store(int(rng.integers(1, 200)))])
    plan = check(segs, 2, 3, 37, share_min=4)
    assert plan["shared_tiles"] > 0
    # the 127-token member can never be shared; ragged tails stay in the stream
    for u in plan["units"]:
        assert u.n_tiles * 128 <= 1000


def test_same_cartridge_twice_in_one_request_and_suffix_free_requests():
    a = Arena(2)
    c = a.store(256)
    segs = [[c, c], [c], [c, a.store(5)], [c]]
    plan = check(segs, 2, 4, 16, share_min=2)
    assert len(plan["readers"]) == 5 and plan["total_tiles"] == 2
    # requests 1 and 3 have no stream token at all: their row groups are merged from shared partials only
    rgs = {m.row_group for m in plan["merges"]}
    assert {2, 3, 6, 7} <= rgs


def test_more_readers_than_one_m_tile_holds():
    a = Arena(1)
    c = a.store(640)
    segs = [[c, a.store(3)] for _ in range(50)]
    plan = check(segs, 1, 8, 20, share_min=4)          # 16 readers per M-tile -> 4 M-tiles (16,16,16,2)
    assert sorted({(u.reader_begin, u.n_readers) for u in plan["units"]}) == [(0, 16), (16, 16), (32, 16), (48, 2)]


def test_below_the_reader_threshold_nothing_is_shared():
    a = Arena(2)
    c = a.store(1024)
    segs = [[c, a.store(10)] for _ in range(3)]
    plan = check(segs, 2, 4, 8, share_min=4)
    assert not plan["units"] and plan["n_unit_cta_used"] == 0 and plan["shared_tiles"] == 0
    old = binding.cart_plan_build(segs, 2, 8, 64)
    assert [(i.k_row, i.n_tok, i.flags, i.slot) for i in plan["items"]] == \
           [(i.k_row, i.n_tok, i.flags, i.slot) for i in old["items"]]


def test_sharing_switched_off_equals_the_stream_planner():
    a = Arena(2)
    c = a.store(1024)
    segs = [[c, a.store(10 + i)] for i in range(9)]
    plan = check(segs, 2, 4, 8, share_min=0)
    old = binding.cart_plan_build(segs, 2, 8, 64)
    assert not plan["units"]
    assert [(i.k_row, i.v_row, i.n_tok, i.flags, i.slot, i.merge) for i in plan["items"]] == \
           [(i.k_row, i.v_row, i.n_tok, i.flags, i.slot, i.merge) for i in old["items"]]
    assert plan["cta_begin"] == old["cta_begin"]


def test_few_partial_slots_make_the_shared_ranges_longer_or_switch_sharing_off():
    a = Arena(1)
    c = a.store(128 * 40)
    segs = [[c, a.store(7)] for _ in range(8)]
    roomy = check(segs, 1, 4, 16, share_min=4)
    assert roomy["n_unit_cta_used"] == 16
    tight = check(segs, 1, 4, 16, share_min=4, slots_cap=8 + 32 + 8 * 4)   # room for 4 chunks per reader
    assert 0 < tight["n_unit_cta_used"] <= 4
    none = check(segs, 1, 4, 16, share_min=4, slots_cap=8 + 32 + 4)        # not even one chunk each
    assert none["n_unit_cta_used"] == 0 and not none["units"]


@pytest.mark.parametrize("w", [synth.config3(), synth.config4()])
def test_benchmark_shapes_with_sharing(w):
    a = Arena(w.n_kv_heads)
    carts = [a.store(w.p) for _ in range(w.n_cartridges)]
    suffix = w.suffix_lengths()
    segs = [[carts[c] for c in parts] + [a.store(int(suffix[b]) + 64)] for b, parts in enumerate(w.request_parts())]
    G = w.n_q_heads // w.n_kv_heads
    plan = check(segs, w.n_kv_heads, G, 148)
    assert plan["n_unit_cta_used"] == 148 and plan["n_cta_used"] == 148
    per_rg = plan["n_slots"] / (w.batch * w.n_kv_heads)
    assert per_rg < 10          # what the library's scratch is sized for


@pytest.mark.parametrize("piece_cost", [1, 3, 8])
def test_blocks_balanced_by_tiles_and_pieces(piece_cost):
    # many short suffixes next to a few long ones: by tiles alone some blocks would hold 20 pieces, others 4
    a = Arena(8)
    cart = a.store(4096)
    rng = np.random.default_rng(11)
    segs = [[cart, a.store(int(n))] for n in rng.integers(1, 1025, size=128)]
    plan = check(segs, 8, 4, 148, piece_cost=piece_cost)
    assert plan["n_cta_used"] >= 140
    flat = check([[a.store(int(n))] for n in rng.integers(1, 300, size=40)], 2, 4, 37, share_min=0, piece_cost=piece_cost)
    assert flat["n_cta_used"] >= 25      # a boundary that falls between row groups saves the piece it was charged for


@pytest.mark.parametrize("w", [synth.config3(), synth.config4()])
def test_shared_blocks_balanced_by_tiles_and_units(w):
    a = Arena(w.n_kv_heads)
    carts = [a.store(w.p) for _ in range(w.n_cartridges)]
    suffix = w.suffix_lengths()
    segs = [[carts[c] for c in parts] + [a.store(int(suffix[b]) + 64)] for b, parts in enumerate(w.request_parts())]
    G = w.n_q_heads // w.n_kv_heads
    flat = check(segs, w.n_kv_heads, G, 148)
    plan = check(segs, w.n_kv_heads, G, 148, piece_cost=3, unit_cost=4)
    assert plan["n_unit_cta_used"] >= 140
    # charging for units makes the planner cut fewer runs in two
    assert len(plan["units"]) <= len(flat["units"])


@pytest.mark.parametrize("w", [synth.config3(), synth.config4()])
def test_side_by_side_divides_the_blocks_between_the_two_kernels(w):
    a = Arena(w.n_kv_heads)
    carts = [a.store(w.p) for _ in range(w.n_cartridges)]
    suffix = w.suffix_lengths()
    segs = [[carts[c] for c in parts] + [a.store(int(suffix[b]) + 64)] for b, parts in enumerate(w.request_parts())]
    G = w.n_q_heads // w.n_kv_heads
    plan = check(segs, w.n_kv_heads, G, 148, piece_cost=3, unit_cost=4, side_by_side=1)
    S = plan["n_shared_ctas"]
    if w.cartridges == "shared":
        # one long Cartridge and long suffixes: a quarter of the blocks or so for the tensor-core kernel, and a
        # division that leaves the 32 (M-tile, KV head) runs whole
        assert 16 <= S <= 64 and len(plan["units"]) == 32
        assert plan["n_unit_cta_used"] >= S - 2 and plan["n_cta_used"] >= 148 - S - 2
    else:
        # many short runs: the estimate does not favour either order by the required margin
        assert S == 0 or plan["n_unit_cta_used"] >= S - 2
    forced = check(segs, w.n_kv_heads, G, 148, piece_cost=3, unit_cost=4, side_by_side=50)
    assert forced["n_shared_ctas"] == 50
    # a batch without a shared part, or without a stream part, keeps all blocks for the one kernel
    alone = check([[a.store(300)] for _ in range(9)], w.n_kv_heads, G, 148, side_by_side=1)
    assert alone["n_shared_ctas"] == 0 and alone["n_cta_used"] == 148
    only_shared = check([[carts[0]] for _ in range(8)], w.n_kv_heads, G, 148, side_by_side=1) if w.p % 128 == 0 else None
    if only_shared is not None:
        assert only_shared["n_shared_ctas"] == 0 and not only_shared["items"] and only_shared["n_unit_cta_used"] >= 60


@pytest.mark.parametrize("seed", range(40))
def test_random_batches_keep_every_invariant(seed):
    """Random pools, compositions, suffix lengths, block counts and cost constants: coverage, slot
    bookkeeping and balance must hold for all of them."""
    rng = np.random.default_rng(1000 + seed)
    Hkv = int(rng.choice([1, 2, 8]))
    G = int(rng.choice([1, 3, 4, 8]))
    a = Arena(Hkv)
    pool = [a.store(int(rng.choice([1, 63, 64, 127, 128, 129, 300, 513, 1024, 2048]))) for _ in range(int(rng.integers(1, 5)))]
    n_reqs = int(rng.integers(1, 40))
    segs = []
    for _ in range(n_reqs):
        k = int(rng.integers(0, min(3, len(pool)) + 1))
        parts = [pool[int(i)] for i in rng.choice(len(pool), k, replace=bool(rng.integers(0, 2)) or k > len(pool))] if k else []
        n_suffix = int(rng.choice([0, 1, 5, 64, 65, 200, 700]))
        r = list(parts)
        if n_suffix or not r:
            r.append(a.store(max(n_suffix, 1), cap_pad=int(rng.integers(0, 70))))
        segs.append(r)
    n_cta = int(rng.choice([1, 2, 7, 37, 148]))
    check(segs, Hkv, G, n_cta, share_min=int(rng.choice([0, 2, 4])), piece_cost=int(rng.choice([0, 1, 3, 9])),
          unit_cost=int(rng.choice([0, 2, 4])), side_by_side=int(rng.choice([0, 1, 1, 5, 40])))
