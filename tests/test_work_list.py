"""Host logic of the backward kernel's work distribution (no GPU): every (key tile, head) item is given to
exactly one CTA, heavy items come before light ones within a chunk, chunks keep a bounded set of heads in
flight, and the loads of the CTAs stay close to the mean."""
import pytest

from paper_2608_00029_b200 import nova_attn as na

SHAPES = [
    # BH, T, D, causal
    (96, 1024, 64, True),      # GPT-2 small: one chunk
    (384, 1024, 64, True),     # large batch: several chunks
    (192, 2048, 64, False),
    (512, 512, 128, True),
    (512, 1024, 128, True),
    (24, 8192, 128, True),     # long context
    (1, 1, 64, True),
    (3, 200, 128, False),      # fewer items than CTAs
    (150, 129, 64, True),      # ragged last tile, chunk smaller than a pass
    (1000, 300, 64, True),
]


def _lists(BH, T, D, causal, n_ctas):
    lists, plan = [], None
    for cta in range(n_ctas):
        items, plan = na.nova_attn_bwd_work_list(BH, T, D, causal, n_ctas, cta)
        lists.append(items)
    return lists, plan


@pytest.mark.parametrize("BH,T,D,causal", SHAPES)
@pytest.mark.parametrize("n_ctas", [148, 132, 7])
def test_every_item_exactly_once_and_balanced(BH, T, D, causal, n_ctas):
    n_tiles = (T + 127) // 128
    lists, (chunk, n_chunks, ppc, plast) = _lists(BH, T, D, causal, n_ctas)
    seen = {}
    for cta, items in enumerate(lists):
        for kt, bh in items:
            assert 0 <= kt < n_tiles and 0 <= bh < BH
            assert (kt, bh) not in seen, f"item {(kt, bh)} on CTAs {seen[(kt, bh)]} and {cta}"
            seen[(kt, bh)] = cta
    assert len(seen) == BH * n_tiles
    # plan consistency
    assert 1 <= chunk <= BH and n_chunks == -(-BH // chunk)
    grid = min(n_ctas, BH * n_tiles)
    assert ppc == -(-chunk * n_tiles // grid)
    assert plast == -(-(BH - (n_chunks - 1) * chunk) * n_tiles // grid)
    # chunks are processed one after the other on every CTA, heaviest key tiles first within a chunk
    for items in lists:
        chunks = [bh // chunk for _, bh in items]
        assert chunks == sorted(chunks)
        for c in set(chunks):
            kts = [kt for kt, bh in items if bh // chunk == c]
            assert kts == sorted(kts)
    # load balance: tiles per CTA (a causal item of key tile kt visits n_tiles - kt query tiles)
    w = [sum((n_tiles - kt) if causal else n_tiles for kt, _ in items) for items in lists[:grid]]
    heaviest = n_tiles
    assert max(w) - sum(w) / len(w) <= 1.01 * heaviest + 0.08 * sum(w) / len(w)


def test_chunks_bound_the_heads_in_flight():
    # B=16, H=32, T=1024, D=128: 1.5 MB of accumulator and inputs per head; a chunk stays below about 64 MB
    _, (chunk, n_chunks, ppc, _) = _lists(512, 1024, 128, True, 148)
    assert n_chunks > 1 and chunk * 1024 * 128 * 12 <= 64 << 20 and ppc >= 2
    # the GPT-2-small shape fits as a whole
    _, (chunk, n_chunks, _, _) = _lists(96, 1024, 64, True, 148)
    assert (chunk, n_chunks) == (96, 1)


def test_bad_arguments():
    for args in [(0, 128, 64, True, 148, 0), (4, 0, 64, True, 148, 0), (4, 128, 96, True, 148, 0),
                 (4, 128, 64, True, 0, 0), (4, 128, 64, True, 148, 148), (4, 128, 64, True, 148, -1)]:
        with pytest.raises(na.NovaAttnError) as ei:
            na.nova_attn_bwd_work_list(*args)
        assert ei.value.status == na.ERR_SHAPE


def test_random_shapes_cover_every_item_once():
    """Seeded random problems, including ones with many small heads and with more CTAs than items."""
    import random
    rng = random.Random(7)
    for _ in range(40):
        BH = rng.choice([1, 2, 5, 17, 96, 200, 777, 3000])
        T = rng.choice([1, 127, 128, 129, 640, 1500, 4096, 20000])
        D = rng.choice([64, 128])
        causal = rng.random() < 0.7
        n_ctas = rng.choice([1, 3, 64, 148, 160])
        n_tiles = (T + 127) // 128
        if BH * n_tiles > 40000:
            continue
        seen = set()
        loads = []
        for cta in range(n_ctas):
            items, (chunk, n_chunks, _, _) = na.nova_attn_bwd_work_list(BH, T, D, causal, n_ctas, cta)
            assert 1 <= chunk <= BH and n_chunks == -(-BH // chunk)
            for it in items:
                assert it not in seen
                seen.add(it)
            loads.append(sum((n_tiles - kt) if causal else n_tiles for kt, _ in items))
        assert len(seen) == BH * n_tiles, (BH, T, D, causal, n_ctas)
        assert all(0 <= kt < n_tiles and 0 <= bh < BH for kt, bh in seen)
        grid = min(n_ctas, BH * n_tiles)
        mean = sum(loads) / grid
        # no CTA carries more than the mean plus one heaviest item and a tenth
        assert max(loads) <= mean * 1.1 + n_tiles, (BH, T, D, causal, n_ctas, max(loads), mean)
