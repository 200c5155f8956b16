"""The flattened tile schedule, replayed on the host through the C ABI: every tile
is handed out exactly once, and the partial-result bookkeeping the combine step
relies on (first slot, last block, skipped empty blocks) is consistent."""
import pytest
import torch

from paper_2211_05102_b200 import binding, build


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()


CASES = [
    ([128, 128], 128, 64, 4),
    ([2048] * 8, 2048, 128, 148),
    ([2048] * 64, 2048, 128, 148),
    ([1, 0, 5, 0, 0, 700, 64, 65, 129, 0], 700, 64, 7),
    ([0, 0, 0], 100, 64, 3),
    ([1], 1, 64, 592),
    ([32768, 1, 17, 20000, 333], 32768, 128, 148),
    ([5] * 1000, 64, 64, 148),
    ([300, -4, 9999], 512, 128, 5),
]


@pytest.mark.parametrize("lengths,Lmax,tile,G", CASES)
def test_schedule_partitions_the_tiles(lengths, Lmax, tile, G):
    ln = torch.tensor(lengths, dtype=torch.int32)
    nt = [(min(max(x, 0), Lmax) + tile - 1) // tile for x in lengths]
    T = sum(nt)
    covered = {b: [] for b in range(len(lengths))}
    info = {}
    parts = {b: [] for b in range(len(lengths))}
    spans = [(i * T // G, (i + 1) * T // G) for i in range(G)]
    for cta in range(G):
        segs = binding.mqa_debug_schedule(ln, Lmax, tile, G, cta)
        assert sum(t1 - t0 for _, t0, t1, *_ in segs) == spans[cta][1] - spans[cta][0]
        slots_used = set()
        for (b, t0, t1, whole, slot, owns_first, last_cta) in segs:
            assert 0 <= t0 < t1 <= nt[b]
            covered[b].append((t0, t1))
            assert whole == int(t0 == 0 and t1 == nt[b])
            if whole:
                assert slot == -1
            else:
                assert slot in (2 * cta, 2 * cta + 1) and slot not in slots_used
                slots_used.add(slot)
                parts[b].append((cta, slot))
            if owns_first:
                assert t0 == 0
                info[b] = (slot, last_cta)
    for b, n in enumerate(nt):
        segs = sorted(covered[b])
        if n == 0:
            assert segs == [] and b not in info
            continue
        assert segs[0][0] == 0 and segs[-1][1] == n
        for (a0, a1), (b0, b1) in zip(segs[:-1], segs[1:]):
            assert a1 == b0
        # the combine step's enumeration of this sequence's partial results
        first_slot, last_cta = info[b]
        if first_slot < 0:
            assert parts[b] == []
            continue
        expect = [first_slot] + [2 * i for i in range(first_slot // 2 + 1, last_cta + 1)
                                 if spans[i][0] != spans[i][1]]
        assert [s for _, s in sorted(parts[b])] == expect


def test_uniform_ctas_keeps_cuts_on_sequence_boundaries():
    """The split-count heuristic for uniform batches: it never asks for more blocks than the plan has, and
    whatever smaller count it picks either takes whole sequences per block or cuts every sequence into the
    same number of equal parts."""
    for B in list(range(1, 70)) + [96, 100, 128, 148, 200, 256, 296, 300, 444, 500, 512, 1000, 1024, 4096]:
        for nt in (1, 2, 3, 4, 7, 8, 12, 16, 64, 256):
            for G in (1, 7, 128, 132, 148, 592):
                g = binding.mqa_uniform_ctas(B, nt, G)
                assert 1 <= g <= G
                if g != G:
                    whole = B % g == 0
                    equal_parts = g % B == 0 and nt % (g // B) == 0
                    assert whole or equal_parts, (B, nt, G, g)
                if B * nt <= G or nt == 1:
                    assert g == G     # one tile per block or per sequence: nothing to align


def test_uniform_ctas_on_the_named_shapes():
    # 512 sequences of 16 tiles on 148 SMs: 4 whole sequences per block
    assert binding.mqa_uniform_ctas(512, 16, 148) == 128
    # 64 sequences of 16 tiles: every sequence in two halves
    assert binding.mqa_uniform_ctas(64, 16, 148) == 128
    # no near divisor: the even share of the flattened tiles stays
    assert binding.mqa_uniform_ctas(300, 8, 148) == 148
    assert binding.mqa_uniform_ctas(200, 16, 148) == 148
    with pytest.raises(binding.MqaError):
        binding.mqa_uniform_ctas(0, 16, 148)


@pytest.mark.parametrize("B,nt,G", [(512, 16, 148), (64, 16, 148), (160, 2, 148), (50, 4, 148), (32, 64, 148)])
def test_aligned_block_count_has_no_ragged_cut(B, nt, G):
    """Replay the schedule at the chosen block count: blocks hold whole sequences only, or every sequence is
    cut into parts of equal size."""
    g = binding.mqa_uniform_ctas(B, nt, G)
    assert g < G
    ln = torch.full((B,), nt * 128, dtype=torch.int32)
    sizes = set()
    for cta in range(g):
        for (b, t0, t1, whole, slot, owns_first, last_cta) in binding.mqa_debug_schedule(ln, nt * 128, 128, g, cta):
            sizes.add(t1 - t0)
    assert len(sizes) == 1 and nt % sizes.pop() == 0
