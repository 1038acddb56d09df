"""The item-to-CTA mapping of the segment-gated LoRA GEMM, checked on the CPU (no GPU needed).

The fused layer hands blocks of its intermediate t from the CTAs that compute them to the CTAs that read them.
Forward progress must not depend on the whole grid being resident, so the producers of t have to be the CTAs the
hardware starts first (the lowest block indices) and must never wait before they publish.  The mapping is a
host/device function of the shape alone; the library exposes it through a host-only entry point.
"""
import numpy as np
import pytest

from paper_2604_11035_b200.binding import lora_work_item

SHAPES = [  # (m, n, rank): model-sized layer, wide layer, rank 1024, ragged shapes, one-CTA fused form, two-launch form
    (3840, 4096, 128), (3840, 12288, 128), (3840, 4096, 1024), (517, 544, 192), (300, 544, 512), (700, 1120, 64),
    (6200, 288, 768), (6200, 544, 320), (128, 32, 64), (20000, 4096, 128)]


def _plan(m, n, rank, sms=148):
    first = lora_work_item(m, n, rank, sms, 0, 0)
    units = first["units"]
    items = []
    for u in range(units):
        k = lora_work_item(m, n, rank, sms, u, 0)["n_items"]
        items.append([lora_work_item(m, n, rank, sms, u, i) for i in range(k)])
    return first, items


@pytest.mark.parametrize("m,n,rank", SHAPES)
def test_every_output_element_is_computed_exactly_once(m, n, rank):
    first, items = _plan(m, n, rank)
    cover = np.zeros((m, n), np.int32)
    for unit in items:
        for it in unit:
            if it["pre"]:
                continue
            r1, c1 = min(m, it["m0"] + it["tile_rows"]), min(n, it["n0"] + it["cols"])
            if it["m0"] < m and it["n0"] < n:
                cover[it["m0"]:r1, it["n0"]:c1] += 1
    assert cover.min() == 1 and cover.max() == 1
    assert first["units"] <= (148 if first["form"] < 2 else 74)


@pytest.mark.parametrize("m,n,rank", SHAPES)
def test_blocks_of_t_are_on_the_lowest_block_indices_and_come_first(m, n, rank):
    first, items = _plan(m, n, rank)
    if first["form"] == 0:                       # two launches: no block of t inside the launch that writes y
        assert not any(it["pre"] for unit in items for it in unit)
        return
    pre_units = [u for u, unit in enumerate(items) if any(it["pre"] for it in unit)]
    # the producers are exactly the first units in block-index order ...
    assert pre_units == list(range(len(pre_units))) and len(pre_units) > 0
    # ... each starts with its block (it never waits on another unit before it publishes) ...
    for u in pre_units:
        assert items[u][0]["pre"] == 1 and sum(it["pre"] for it in items[u]) == 1
    # ... the blocks tile t exactly once ...
    cover = np.zeros((m, rank), np.int32)
    for u in pre_units:
        it = items[u][0]
        cover[it["m0"]:min(m, it["m0"] + it["tile_rows"]), it["n0"]:it["n0"] + it["cols"]] += 1
    assert cover.min() == 1 and cover.max() == 1
    # ... and the producers are the units with the fewest output tiles (they carry the extra block)
    out_items = [sum(1 - it["pre"] for it in unit) for unit in items]
    assert max(out_items[u] for u in pre_units) <= min(out_items[len(pre_units):] or [10 ** 9])


def test_forms_are_chosen_by_shape_alone():
    assert lora_work_item(3840, 4096, 128, 148, 0, 0)["form"] == 2      # CTA pairs
    assert lora_work_item(6200, 288, 768, 148, 0, 0)["form"] == 1       # more blocks of t than pairs: one-CTA kernel
    assert lora_work_item(6200, 544, 320, 148, 0, 0)["form"] == 0       # rank neither <= 256 nor a multiple of it
