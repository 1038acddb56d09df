"""Launch shape of the verification kernels (host logic, no GPU): how many CTAs a row of the first pass and a
sampled row of the second pass are cut into for a batch on a GPU of a given size."""
import itertools

import pytest

from paper_2604_11035_b200.binding import verify_grid

V = 151936
SMS = 148


@pytest.mark.parametrize("batch,stride,propose_mode",
                         list(itertools.product([1, 2, 8, 32, 64, 148, 256, 512], [2, 4, 8, 16], [0, 1])))
def test_pieces_are_bounded_and_fill_the_machine(batch, stride, propose_mode):
    g = verify_grid(batch, stride, V, propose_mode, SMS)
    rows = batch * (2 * stride - 1)
    sampled = batch * (stride if propose_mode == 0 else 1)
    assert 1 <= g["row_splits"] <= 16 and 4 <= g["sample_splits"] <= 16
    assert g["row_ctas"] == rows * g["row_splits"] and g["sample_ctas"] == sampled * g["sample_splits"]
    # a piece keeps at least 8k elements
    assert V // g["row_splits"] >= 8192 and V // g["sample_splits"] >= 8192
    # first pass: the machine is filled (four CTAs per SM) unless sixteen pieces per row cannot do it
    assert g["row_ctas"] >= min(4 * SMS, 16 * rows)
    # one more piece per row is only taken while it is needed to reach that
    if g["row_splits"] > 1:
        assert rows * (g["row_splits"] - 1) < 4 * SMS
    # second pass: more than four pieces only while all CTAs are resident at once (four per SM)
    if g["sample_splits"] > 4:
        assert g["sample_ctas"] <= 4 * SMS


def test_large_batches_take_one_cta_per_row_and_four_pieces_per_draw():
    for batch in (256, 512):
        g = verify_grid(batch, 8, V, 1, SMS)
        assert g["row_splits"] == 1 and g["sample_splits"] == 4


def test_single_sequence_is_cut_as_finely_as_allowed():
    g = verify_grid(1, 8, V, 1, SMS)
    assert g["row_splits"] == 16 and g["sample_splits"] == 16


def test_short_rows_are_not_cut_below_8k_elements():
    g = verify_grid(1, 4, 4096, 1, SMS)
    assert g["row_splits"] == 1 and g["sample_splits"] == 1
    g = verify_grid(1, 4, 32768, 0, SMS)
    assert g["row_splits"] == 4 and g["sample_splits"] == 4


def test_pieces_shrink_as_the_batch_grows():
    prev = None
    for batch in (1, 2, 4, 8, 16, 32, 64, 128, 256, 512):
        g = verify_grid(batch, 8, V, 1, SMS)
        if prev is not None:
            assert g["row_splits"] <= prev["row_splits"] and g["sample_splits"] <= prev["sample_splits"]
        prev = g
